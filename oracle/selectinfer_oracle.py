"""SelectInfer oracle: TEST INFRASTRUCTURE ONLY, never a product path.

Plain CPU statements of every step of the selective-computation hot path, written
from the paper's description and independent of the CUDA library (no shared code,
neither imports the other).  Only tests, the smoke check and the benchmark's
cpu_baseline / reference legs may import this module.

* ``ffn`` / ``ffn_tokens`` / ``ffn_dense_masked`` -- float64 selective SwiGLU FFN on the
  full weights with global neuron ids (C loops in ``si_oracle.c``; Section 3 for the
  neuron <-> weight-slice correspondence, Section 5 for "compute only the selected
  loaded neurons").
* ``ffn_chain`` -- the FFN applied layer after layer (Section 4: the same for every FFN layer), each
  step reading the output of the step before it, rounded to the model's 16-bit type; ``rmsnorm`` is
  the gain-free RMS normalisation in front of the FFN of the paper's pre-norm models and ``round_bits``
  the rounding (both library-pinned).
* ``select_topk`` -- Section 5: sort activations in descending order, keep the top
  alpha, record their indices.  Tie-break (paper silent): lower index wins; +0 == -0;
  NaN ranks below everything.  Output ascending by index.
* ``select_threshold`` -- extension with no counterpart in the paper (brute-force
  pinned only).
* ``prefill_vote`` -- Section 5: per-token top alpha, frequency count over the prompt's tokens,
  top beta by frequency, merge with the static prefix up to phi.
* ``union`` -- sorted set union of per-token lists plus per-token membership bitmasks.
* ``profile_scores`` / ``merge_scores`` / ``ranking`` -- Section 3, Eq. 1: per-neuron sums of absolute
  activations, merged over score files after normalising by token count, ranked by importance.
* ``loadset`` -- Section 4: base = top delta of the task ranking, then the model
  ranking in order, skipping ids already chosen, until gamma neurons are loaded.
* ``shard_slots`` / ``shard_lists`` -- the loaded slots dealt round-robin to P devices and a slot list
  rewritten for one of them.  Section 5 defines the layer output as a sum over the selected neurons, so
  the partial outputs of disjoint neuron subsets add up to it; the paper itself runs on one device.
* ``memory_saving`` -- Eq. 2.
* ``layer_range`` -- Table 1 "first layer 5 / last layer -2".

Pins live in tests/test_oracle_pins.py.  Parity unpinned: the paper's task-accuracy
results (they need its datasets and trained weights); nothing here computes them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "si_oracle.c")
_LIB = os.path.join(_HERE, "libsi_oracle.so")

F64, F16, BF16 = 0, 1, 2
_DTYPES = {"f64": F64, "f16": F16, "bf16": BF16}


def build(force: bool = False) -> str:
    """Compile si_oracle.c with gcc -O2 -fopenmp (no BLAS, no intrinsics)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, ip = ctypes.c_void_p, ctypes.c_int
        lib.so_ffn.argtypes = [vp, vp, vp, ip, ip, ip, vp, vp, ip, vp, vp, ip]
        lib.so_ffn.restype = ip
        lib.so_ffn_dense_masked.argtypes = [vp, vp, vp, ip, ip, ip, vp, vp, vp]
        lib.so_ffn_dense_masked.restype = ip
        lib.so_ffn_tokens.argtypes = [vp, vp, vp, ip, ip, ip, vp, ip, vp, vp, vp, ip]
        lib.so_ffn_tokens.restype = ip
        _lib = lib
    return _lib


def _prep(a, dtype_code):
    want = np.float64 if dtype_code == F64 else np.uint16
    a = np.ascontiguousarray(a)
    if a.dtype != want:
        raise TypeError(f"expected {want} storage for dtype code {dtype_code}, got {a.dtype}")
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def host_threads() -> int:
    return len(os.sched_getaffinity(0))


def ffn(Wg, Wu, Wd, x, A, dtype: str = "f64", threads: int = 1, return_h: bool = False):
    """y[d_model] float64 = selective FFN over global neuron ids A (Sections 3, 5).

    Wg, Wu: [d_ff, d_model]; Wd: [d_model, d_ff]; x: [d_model].  For dtype "f16"/"bf16"
    the arrays hold raw uint16 bit patterns; for "f64" float64 values.
    """
    code = _DTYPES[dtype]
    Wg, Wu, Wd, x = (_prep(a, code) for a in (Wg, Wu, Wd, x))
    d_ff, d_model = Wg.shape
    assert Wu.shape == (d_ff, d_model) and Wd.shape == (d_model, d_ff) and x.shape == (d_model,)
    A = np.ascontiguousarray(A, dtype=np.int32)
    y = np.empty(d_model, dtype=np.float64)
    h = np.empty(max(len(A), 1), dtype=np.float64)
    rc = _load().so_ffn(_ptr(Wg), _ptr(Wu), _ptr(Wd), code, d_ff, d_model, _ptr(x), _ptr(A),
                        len(A), _ptr(y), _ptr(h), threads)
    if rc:
        raise ValueError("neuron ids must be distinct and in [0, d_ff)")
    return (y, h[: len(A)]) if return_h else y


def ffn_dense_masked(Wg, Wu, Wd, x, keep, dtype: str = "f64"):
    """Dense FFN over all neurons with h_i zeroed where keep[i] == 0 (brute force)."""
    code = _DTYPES[dtype]
    Wg, Wu, Wd, x = (_prep(a, code) for a in (Wg, Wu, Wd, x))
    d_ff, d_model = Wg.shape
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    assert keep.shape == (d_ff,)
    y = np.empty(d_model, dtype=np.float64)
    _load().so_ffn_dense_masked(_ptr(Wg), _ptr(Wu), _ptr(Wd), code, d_ff, d_model, _ptr(x),
                                _ptr(keep), _ptr(y))
    return y


def ffn_tokens(Wg, Wu, Wd, X, lists, dtype: str = "f64", threads: int = 1):
    """Y[T, d_model]: token t uses exactly lists[t] (masked-union semantics)."""
    code = _DTYPES[dtype]
    Wg, Wu, Wd, X = (_prep(a, code) for a in (Wg, Wu, Wd, X))
    d_ff, d_model = Wg.shape
    T = X.shape[0]
    assert X.shape == (T, d_model) and len(lists) == T
    offsets = np.zeros(T + 1, dtype=np.int32)
    offsets[1:] = np.cumsum([len(l) for l in lists])
    flat = (np.concatenate([np.asarray(l, dtype=np.int32) for l in lists])
            if offsets[-1] else np.zeros(1, dtype=np.int32))
    flat = np.ascontiguousarray(flat, dtype=np.int32)
    Y = np.empty((T, d_model), dtype=np.float64)
    rc = _load().so_ffn_tokens(_ptr(Wg), _ptr(Wu), _ptr(Wd), code, d_ff, d_model, _ptr(X), T,
                               _ptr(flat), _ptr(offsets), _ptr(Y), threads)
    if rc:
        raise ValueError("neuron ids must be distinct and in [0, d_ff)")
    return Y


# --------------------------------------------------------------------------- chained layers

def round_bits(v, dtype: str) -> np.ndarray:
    """float64 values -> fp16 / bf16 bit patterns, round to nearest even (through float32, as a model
    that keeps its hidden state in a 16-bit type does)."""
    f = np.asarray(v, dtype=np.float64).astype(np.float32)
    if dtype == "f16":
        return f.astype(np.float16).view(np.uint16)
    u = f.view(np.uint32).astype(np.uint64)
    nan = np.isnan(f)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    r[nan] = 0x7FC0
    return r


def widen_bits(bits, dtype: str) -> np.ndarray:
    """fp16 / bf16 bit patterns -> float64 (exact)."""
    b = np.asarray(bits, dtype=np.uint16)
    if dtype == "f16":
        return b.view(np.float16).astype(np.float64)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rmsnorm(x, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) in float64: the normalisation a pre-norm transformer block applies in
    front of its FFN, without the learned gain."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x) + float(eps))


def ffn_chain(layer_weights, layers, ids, lists, x0_bits, dtype: str, residual: bool = False, prenorm: bool = False,
              eps: float = 0.0, threads: int = 1):
    """One chain: step s runs the selective FFN of layer layers[s] (weights layer_weights[layers[s]],
    global ids ids[layers[s]][lists[s]]) on the output of step s - 1; step 0 reads x0.  Per step:
        in   = x0 or the rounded output of the step before          (16-bit)
        xn   = round(rmsnorm(in))  if prenorm  else  in             (16-bit: what the dot products see)
        out  = round((in if residual else 0) + FFN(xn))             (16-bit: what the next step reads)
    Returns (out bits [steps, d], xn bits [steps, d], float64 outputs before rounding [steps, d])."""
    cur = np.asarray(x0_bits, dtype=np.uint16)
    outs, xns, raws = [], [], []
    for s, layer in enumerate(layers):
        xin = widen_bits(cur, dtype)
        xn_bits = round_bits(rmsnorm(xin, eps), dtype) if prenorm else cur
        wg, wu, wd = layer_weights[layer]
        gids = np.asarray(ids[layer])[np.asarray(lists[s], dtype=np.int64)] if len(lists[s]) else np.zeros(0, np.int32)
        y = ffn(wg, wu, wd, xn_bits, gids, dtype=dtype, threads=threads)
        if residual:
            y = y + xin
        cur = round_bits(y, dtype)
        outs.append(cur); xns.append(xn_bits); raws.append(y)
    return np.stack(outs), np.stack(xns), np.stack(raws)


# --------------------------------------------------------------------------- selection

def _rank_order(scores: np.ndarray, use_abs: bool):
    """Indices ordered by (score descending, index ascending); NaN last; +0 == -0."""
    s = np.asarray(scores, dtype=np.float32)
    if use_abs:
        s = np.abs(s)
    order = []
    for i, v in enumerate(s.tolist()):       # python floats: exact images of the float32s
        is_nan = v != v
        order.append((1 if is_nan else 0, 0.0 if is_nan else -v, i))
    order.sort()                             # -0.0 == 0.0 compares equal, index breaks the tie
    return [i for _, _, i in order]


def select_topk(scores, k: int, use_abs: bool = False) -> np.ndarray:
    """Section 5: top-k indices of the scores, returned ascending by index."""
    n = len(scores)
    if not 0 <= k <= n:
        raise ValueError("k out of range")
    chosen = _rank_order(scores, use_abs)[:k]
    return np.array(sorted(chosen), dtype=np.int32)


def select_threshold(scores, tau: float, use_abs: bool = False) -> np.ndarray:
    """Extension (not in the paper): indices with score > tau, NaN excluded, ascending."""
    s = np.asarray(scores, dtype=np.float32)
    if use_abs:
        s = np.abs(s)
    tau32 = np.float32(tau)
    return np.array([i for i, v in enumerate(s) if v > tau32], dtype=np.int32)


def prefill_vote(acts, alpha: int, beta: int, n_static: int, phi_count: int, use_abs: bool = True):
    """Section 5, selection of the dynamic neurons during prefill, in the paper's order:

    1. for every prompt token, rank the activations of all loaded neurons in descending order and
       record the indices of the top alpha (``select_topk``: ties to the lower index);
    2. count how often each neuron occurs in these lists;
    3. the beta neurons with the highest frequency are the dynamic candidates (ties: lower slot;
       a neuron that occurs in no list is never a candidate -- reading, the paper is silent);
    4. the static neurons (slots 0 .. n_static-1: the base neurons come first in the store) are
       combined with the candidates, walked in order of frequency, candidates that are already
       static skipped, until phi_count neurons are chosen.

    acts: [T, n] activations h_i(x_t) of the n loaded neurons.  use_abs ranks |a| (the paper's
    profiling and overlap studies define "most active" by the absolute value; its run-time text
    says only "descending order").  Returns (chosen slots ascending, int64 counts [n]).
    """
    a = np.asarray(acts, dtype=np.float32)
    T, n = a.shape
    if not (0 <= alpha <= n and 0 <= beta <= n and 0 <= n_static <= n and 0 <= phi_count <= n):
        raise ValueError("count out of range")
    counts = np.zeros(n, dtype=np.int64)
    for t in range(T):
        for i in select_topk(a[t], alpha, use_abs=use_abs):
            counts[i] += 1
    by_frequency = sorted(range(n), key=lambda i: (-int(counts[i]), i))
    candidates = [i for i in by_frequency[:beta] if counts[i] > 0]
    chosen = list(range(min(n_static, phi_count)))
    for i in candidates:
        if len(chosen) >= phi_count:
            break
        if i >= n_static:
            chosen.append(i)
    return np.array(sorted(chosen), dtype=np.int32), counts


def union(lists, n_loaded: int):
    """Sorted union U of the lists, per-token bitmasks over positions in U, overlap ratios.

    mask[t, p >> 5] bit (p & 31) is set iff U[p] is in lists[t].
    overlap = 1 - |U| / sum_t |A_t|; coverage = |U| / n_loaded.
    """
    seen = set()
    for l in lists:
        seen.update(int(v) for v in l)
    U = np.array(sorted(seen), dtype=np.int32)
    pos = {int(v): p for p, v in enumerate(U)}
    words = (len(U) + 31) // 32
    mask = np.zeros((len(lists), max(words, 1)), dtype=np.uint32)
    total = 0
    for t, l in enumerate(lists):
        for v in l:
            p = pos[int(v)]
            mask[t, p >> 5] |= np.uint32(1 << (p & 31))
            total += 1
    overlap = 1.0 - len(U) / total if total else 0.0
    return U, mask[:, :words], overlap, len(U) / n_loaded


def loadset(task_rank, model_rank, n_base: int, n_loaded: int) -> np.ndarray:
    """Section 4: base neurons first (top n_base of the task ranking), then secondary
    neurons from the model ranking, skipping those already chosen, until n_loaded."""
    out = [int(v) for v in task_rank[:n_base]]
    chosen = set(out)
    for v in model_rank:
        if len(out) >= n_loaded:
            break
        v = int(v)
        if v not in chosen:
            chosen.add(v)
            out.append(v)
    if len(out) != n_loaded:
        raise ValueError("rankings too short for n_loaded")
    return np.array(out, dtype=np.int32)


def profile_scores(acts, scores=None) -> np.ndarray:
    """Eq. 1: s_n = sum over the processed tokens t of |a_n(t)|.  acts: [T, n] float32 activations;
    scores: running float64 totals of earlier prompts (added to, tokens in order) or None."""
    a = np.asarray(acts, dtype=np.float32)
    out = np.zeros(a.shape[1], dtype=np.float64) if scores is None else np.array(scores, dtype=np.float64)
    for t in range(a.shape[0]):                  # token by token, in order
        out += np.abs(a[t]).astype(np.float64)
    return out


def merge_scores(files) -> np.ndarray:
    """Section 3: score files are merged by normalising each file's scores by its token count and
    summing the normalised values.  files: sequence of (scores float64 [n], tokens), added in order."""
    merged = None
    for scores, tokens in files:
        if tokens <= 0:
            raise ValueError("token count must be positive")
        part = np.asarray(scores, dtype=np.float64) / float(tokens)
        merged = part if merged is None else merged + part
    return merged


def ranking(scores) -> np.ndarray:
    """Section 3: neuron indices in decreasing order of importance (ties: lower index first; NaN last)."""
    s = np.asarray(scores, dtype=np.float64)
    key = [(1 if v != v else 0, 0.0 if v != v else -v, i) for i, v in enumerate(s.tolist())]
    key.sort()
    return np.array([i for _, _, i in key], dtype=np.int32)


def shard_slots(n_loaded: int, rank: int, world: int) -> np.ndarray:
    """Global slots owned by device `rank` of `world`: rank, rank + world, ...  (local slot j = global
    slot rank + j * world, so every device keeps the importance order and a share of the hot slots)."""
    return np.arange(rank, n_loaded, world, dtype=np.int32)


def shard_lists(lists, rank: int, world: int):
    """Each list restricted to the slots device `rank` owns, as local slot numbers, order kept."""
    out = []
    for l in lists:
        l = np.asarray(l, dtype=np.int64)
        out.append((l[l % world == rank] // world).astype(np.int32))
    return out


def memory_saving(n_ffn_params: float, r_load: float, r_layer: float, bytes_per_param: float):
    """Eq. 2: bytes saved = N_ffn * (1 - r_load) * r_layer * s."""
    return n_ffn_params * (1.0 - r_load) * r_layer * bytes_per_param


def layer_range(n_layers: int, first: int = 5, last: int = -2):
    """Table 1: selective layers = first ... n_layers + last - 1 (0-based)."""
    return list(range(first, n_layers + last))


def count_from_pct(pct: int, n: int) -> int:
    """Fractions -> counts: floor(pct * n / 100) in integers."""
    return (pct * n) // 100


def error_metrics(y, y_ref):
    """(max|err| / max|y_ref|, mean|err| / mean|y_ref|) for one token."""
    y = np.asarray(y, dtype=np.float64)
    y_ref = np.asarray(y_ref, dtype=np.float64)
    err = np.abs(y - y_ref)
    mx = np.max(np.abs(y_ref))
    mn = np.mean(np.abs(y_ref))
    return (float(np.max(err) / mx) if mx > 0 else float(np.max(err)),
            float(np.mean(err) / mn) if mn > 0 else float(np.mean(err)))
