"""Helpers for the GPU parity tests: build a store from a synthetic workload and keep the
host copies the oracle needs.  No method arithmetic here."""
import numpy as np
import torch

from paper_2607_18081_b200 import workloads as wl

MAX_ERR = 2e-2      # max|err| <= 2e-2 * max|y_ref|   (per token)
MEAN_REL = 5e-3     # mean|err| / mean|y_ref| <= 5e-3 (per token)
# fp32 outputs of the decode kernels: 16-bit inputs are widened exactly and every product and sum is
# fp32, so the error against float64 is a few fp32 roundings of a sum of up to ~10^4 terms of mixed sign
# (observed ~1e-6 of max|y_ref|).  A dropped column group, record or split shows up at 1e-2 and more.
F32_MAX_ERR = 5e-5
F32_MEAN_REL = 2e-5


def to_dev(bits: np.ndarray, dtype: str) -> torch.Tensor:
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    return torch.from_numpy(bits.view(np.int16)).cuda().view(tdt)


def from_dev(t: torch.Tensor) -> np.ndarray:
    """float64 host copy of a device tensor of any float dtype (exact widening)."""
    return t.detach().to(torch.float64).cpu().numpy()


class LoadedModel:
    def __init__(self, cfg, keep_layers=None, n_layers=None):
        from paper_2607_18081_b200 import api
        self.cfg = cfg
        L = cfg.n_layers if n_layers is None else n_layers
        self.L = L
        keep = set(range(L)) if keep_layers is None else set(keep_layers)
        self.host = {}          # layer -> (wg, wu, wd) uint16
        self.ids = []           # per layer: global ids in slot order
        self.slot_of_rank = []
        self.store = api.NeuronStore(L, cfg.d_model, cfg.d_ff, [cfg.n_loaded] * L, cfg.dtype)
        for l in range(L):
            wg, wu, wd = wl.layer_weights(cfg, l)
            ids, sor = wl.loaded_ids(cfg, l)
            self.ids.append(ids)
            self.slot_of_rank.append(sor)
            self.store.load(l, to_dev(wg, cfg.dtype), to_dev(wu, cfg.dtype), to_dev(wd, cfg.dtype), ids,
                            cfg.n_base)
            if l in keep:
                self.host[l] = (wg, wu, wd)
        torch.cuda.synchronize()

    def oracle_y(self, layer, x_bits, slots, threads=None):
        from oracle import selectinfer_oracle as so
        wg, wu, wd = self.host[layer]
        gids = self.ids[layer][np.asarray(slots, dtype=np.int64)] if len(slots) else np.zeros(0, np.int32)
        return so.ffn(wg, wu, wd, x_bits, gids, dtype=self.cfg.dtype,
                      threads=so.host_threads() if threads is None else threads)


def assert_close(y, y_ref, what=""):
    from oracle import selectinfer_oracle as so
    e_max, e_mean = so.error_metrics(y, y_ref)
    assert e_max <= MAX_ERR and e_mean <= MEAN_REL, f"{what}: max-rel {e_max:.3e}, mean-rel {e_mean:.3e}"
    return e_max, e_mean


def assert_close_f32(y, y_ref, what=""):
    """Tight bound for fp32 outputs of the decode kernels (no 16-bit rounding anywhere on the way)."""
    from oracle import selectinfer_oracle as so
    e_max, e_mean = so.error_metrics(y, y_ref)
    assert e_max <= F32_MAX_ERR and e_mean <= F32_MEAN_REL, f"{what}: max-rel {e_max:.3e}, mean-rel {e_mean:.3e} (fp32 bound)"
    return e_max, e_mean
