"""Seeded synthetic workloads (inputs only -- none of the method's arithmetic lives here).

The five benchmark configurations are FFN-shaped stand-ins for the paper's models
and datasets (Llama-2-7B / Llama-3-8B FFN dimensions; a Zipf activity model standing
in for the stable hot core plus varying tail of Sections 2.2-2.3).  Both the CUDA
library and the CPU oracle read tensors made here; neither imports the other.

Recipe (base seed 20260718, every stream keyed by (seed, config, layer, tag[, token])):
  * weights  ~ N(0, 0.02), rounded nearest-even to fp16 (c1) / bf16 (c2-c5), PyTorch
    [out, in] layout: W_gate, W_up [d_ff, d_model]; W_down [d_model, d_ff];
  * x        ~ N(0, 1) rounded likewise, independent per (layer, token);
  * ranking  pi_l = seeded permutation of 0..d_ff-1 per layer (the synthetic neuron file);
  * loaded   c1: first n_ld ids of a second, independent permutation (slot order), Zipf
             rank = position in pi_l restricted to the loaded set;
             c2-c5: first n_ld ids of pi_l, slot s = rank s; n_base = 30 % of d_ff;
  * active   k distinct slots without replacement with weight (r + 1)^-1.1 for rank r,
             by Gumbel-top-k; passed sorted ascending;
  * scores   ~ N(0, 1) float32 per (layer, token) over the loaded slots (c5 selector);
  * counts   = (pct * N) // 100.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace

import numpy as np

SEED = 20260718
ZIPF_S = 1.1

_HERE = os.path.dirname(os.path.abspath(__file__))
_FILL_SRC = os.path.join(_HERE, "csrc", "workload_fill.c")
_FILL_LIB = os.path.join(_HERE, "libsi_workload_fill.so")

_TAG = {"wg": 1, "wu": 2, "wd": 3, "x": 4, "rank": 5, "loadperm": 6, "active": 7, "scores": 8,
        "taskrank": 9}


def count_pct(pct: int, n: int) -> int:
    return (pct * n) // 100


@dataclass(frozen=True)
class Config:
    name: str
    cfg_id: int
    d_model: int
    d_ff: int
    n_layers: int
    dtype: str            # "f16" | "bf16"
    loaded_pct: int
    active_pct: int       # percent of the LOADED neurons
    tokens: int           # decode steps (or prefill tokens for c4)
    batch: int = 1        # tokens processed together per step
    loaded_rule: str = "rank"   # "rank": first n_ld of pi_l; "perm": independent permutation (c1)
    shared_list: bool = False   # c4: one list per layer = slots 0..k-1

    @property
    def n_loaded(self) -> int:
        return count_pct(self.loaded_pct, self.d_ff)

    @property
    def k_active(self) -> int:
        return count_pct(self.active_pct, self.n_loaded)

    @property
    def n_base(self) -> int:
        return min(count_pct(30, self.d_ff), self.n_loaded)

    @property
    def record_bytes(self) -> int:
        return 3 * self.d_model * 2

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    "c1": Config("c1", 1, 512, 1376, 1, "f16", 50, 25, 16, loaded_rule="perm"),
    "c2": Config("c2", 2, 4096, 11008, 32, "bf16", 70, 20, 128),
    "c3": Config("c3", 3, 4096, 11008, 32, "bf16", 70, 20, 16, batch=4),
    "c4": Config("c4", 4, 4096, 11008, 32, "bf16", 70, 40, 512, batch=512, shared_list=True),
    "c5": Config("c5", 5, 4096, 14336, 32, "bf16", 70, 20, 64),
}
C3_BATCHES = (1, 4, 8, 16, 32)
C5_LOADED = (30, 50, 70, 100)
C5_ACTIVE = (5, 10, 20, 50)


def _seq(cfg: Config, layer: int, tag: str, *extra: int) -> np.random.SeedSequence:
    return np.random.SeedSequence([SEED, cfg.cfg_id, layer, _TAG[tag], *extra])


def _rng(cfg: Config, layer: int, tag: str, *extra: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(_seq(cfg, layer, tag, *extra)))


def _key64(cfg: Config, layer: int, tag: str, *extra: int) -> int:
    return int(_seq(cfg, layer, tag, *extra).generate_state(1, dtype=np.uint64)[0])


_fill = None


def build_fill(force: bool = False) -> str:
    if force or not os.path.exists(_FILL_LIB) or \
            os.path.getmtime(_FILL_LIB) < os.path.getmtime(_FILL_SRC):
        tmp = _FILL_LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp,
                               _FILL_SRC, "-lm"])
        os.replace(tmp, _FILL_LIB)
    return _FILL_LIB


def fill_normal(n: int, std: float, dtype: str, key: int, threads: int | None = None) -> np.ndarray:
    """n samples of N(0, std) as fp16/bf16 bit patterns (uint16)."""
    global _fill
    if _fill is None:
        lib = ctypes.CDLL(build_fill())
        lib.wl_fill_normal.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                       ctypes.c_uint64, ctypes.c_float, ctypes.c_int, ctypes.c_int]
        lib.wl_fill_normal.restype = None
        _fill = lib
    out = np.empty(n, dtype=np.uint16)
    if threads is None:
        threads = len(os.sched_getaffinity(0))
    _fill.wl_fill_normal(out.ctypes.data_as(ctypes.c_void_p), 0, n, key, std,
                         1 if dtype == "f16" else 2, threads)
    return out


def layer_weights(cfg: Config, layer: int):
    """(W_gate [F,d], W_up [F,d], W_down [d,F]) as uint16 bit patterns."""
    F, d = cfg.d_ff, cfg.d_model
    wg = fill_normal(F * d, 0.02, cfg.dtype, _key64(cfg, layer, "wg")).reshape(F, d)
    wu = fill_normal(F * d, 0.02, cfg.dtype, _key64(cfg, layer, "wu")).reshape(F, d)
    wd = fill_normal(F * d, 0.02, cfg.dtype, _key64(cfg, layer, "wd")).reshape(d, F)
    return wg, wu, wd


def x_tokens(cfg: Config, layer: int, tokens: int, first_token: int = 0) -> np.ndarray:
    """x [tokens, d_model] ~ N(0,1) as bit patterns, independent per (layer, token)."""
    out = np.empty((tokens, cfg.d_model), dtype=np.uint16)
    for t in range(tokens):
        out[t] = fill_normal(cfg.d_model, 1.0, cfg.dtype,
                             _key64(cfg, layer, "x", first_token + t), threads=1)
    return out


def ranking(cfg: Config, layer: int) -> np.ndarray:
    """pi_l: neuron ids in decreasing (synthetic) importance."""
    return _rng(cfg, layer, "rank").permutation(cfg.d_ff).astype(np.int32)


def task_ranking(cfg: Config, layer: int) -> np.ndarray:
    """A second, task-specific ranking (used only by the base/secondary loader cases)."""
    return _rng(cfg, layer, "taskrank").permutation(cfg.d_ff).astype(np.int32)


def loaded_ids(cfg: Config, layer: int):
    """(ids int32[n_ld] global neuron ids in slot order, slot_of_rank int32[n_ld])."""
    n_ld = cfg.n_loaded
    pi = ranking(cfg, layer)
    if cfg.loaded_rule == "rank":
        return pi[:n_ld].copy(), np.arange(n_ld, dtype=np.int32)
    sigma = _rng(cfg, layer, "loadperm").permutation(cfg.d_ff).astype(np.int32)
    ids = sigma[:n_ld].copy()
    pos_in_pi = np.empty(cfg.d_ff, dtype=np.int64)
    pos_in_pi[pi] = np.arange(cfg.d_ff)
    slot_of_rank = np.argsort(pos_in_pi[ids], kind="stable").astype(np.int32)
    return ids, slot_of_rank


def zipf_lists(cfg: Config, layer: int, tokens: int, k: int | None = None,
               slot_of_rank: np.ndarray | None = None, first_token: int = 0) -> np.ndarray:
    """[tokens, k] int32 slot lists, each sorted ascending (Gumbel-top-k over Zipf weights)."""
    n_ld = cfg.n_loaded
    k = cfg.k_active if k is None else k
    if cfg.shared_list:
        return np.tile(np.arange(k, dtype=np.int32), (tokens, 1))
    logw = -ZIPF_S * np.log(np.arange(1, n_ld + 1, dtype=np.float64))
    out = np.empty((tokens, k), dtype=np.int32)
    for t in range(tokens):
        g = _rng(cfg, layer, "active", first_token + t).gumbel(size=n_ld)
        keys = logw + g
        ranks = np.argpartition(-keys, k - 1)[:k] if 0 < k < n_ld else np.arange(k)
        slots = ranks if slot_of_rank is None else slot_of_rank[ranks]
        out[t] = np.sort(slots.astype(np.int32))
    return out


def scores(cfg: Config, layer: int, tokens: int, first_token: int = 0) -> np.ndarray:
    """[tokens, n_ld] float32 ~ N(0,1): runtime-selector inputs."""
    out = np.empty((tokens, cfg.n_loaded), dtype=np.float32)
    for t in range(tokens):
        out[t] = _rng(cfg, layer, "scores", first_token + t).standard_normal(
            cfg.n_loaded, dtype=np.float32)
    return out


def selected_bytes_per_token(cfg: Config, k: int | None = None) -> int:
    """Roofline bytes: selected-neuron records only, all layers, one token."""
    k = cfg.k_active if k is None else k
    return k * cfg.record_bytes * cfg.n_layers


def bits_to_float64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of fp16 / bf16 bit patterns (for test-side library cross-checks)."""
    a = np.asarray(a, dtype=np.uint16)
    if dtype == "f16":
        return a.view(np.float16).astype(np.float64)
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def float_to_bits(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round-to-nearest-even float32 -> fp16 / bf16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f16":
        return a.astype(np.float16).view(np.uint16)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)
