"""GPU parity over model shapes other than the benchmark's: hidden sizes of 1024 .. 8192 in both
16-bit types, through every route (single step, stacked steps, union path for a few tokens, the
tensor-core path for many tokens), each token checked against the oracle."""
import numpy as np
import pytest
import torch

from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev

pytestmark = pytest.mark.gpu

# (d_model, d_ff, dtype): d_ff is kept small so that the oracle stays fast; 50 % loaded, 25 % of those active
SHAPES = [
    (1024, 768, "f16"),
    (2048, 1000, "bf16"),
    (3200, 900, "bf16"),      # 400 16-byte chunks per row: a ragged last round of the 256-thread walk
    (4096, 1024, "f16"),
    (5120, 1024, "bf16"),     # three chunks per thread in the persistent kernel, ragged
    (6144, 800, "f16"),       # three full chunks per thread, two ring stages per consumer set
    (7168, 700, "bf16"),      # one consumer set of 512 threads in the persistent kernel, ragged
    (8192, 640, "bf16"),      # the same with full rows
]


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _model(i):
    d, f, dt = SHAPES[i]
    cfg = wl.Config(f"shape{d}", 20 + i, d, f, 2, dt, 50, 25, 8)
    return LoadedModel(cfg)


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


@pytest.mark.parametrize("i", range(len(SHAPES)))
def test_shape_all_routes(api, i):
    m = _model(i)
    cfg = m.cfg
    d, k, L = cfg.d_model, cfg.k_active, 2
    tdt = torch.float16 if cfg.dtype == "f16" else torch.bfloat16

    # ---- one token, one layer per call (per-step kernels) and four stacked steps (persistent kernel)
    steps = 4
    lists = np.stack([wl.zipf_lists(cfg, s % L, 1, slot_of_rank=m.slot_of_rank[s % L])[0] for s in range(steps)])
    x = np.stack([wl.x_tokens(cfg, s % L, 1, first_token=s)[0] for s in range(steps)])
    idx = torch.from_numpy(np.ascontiguousarray(lists, dtype=np.int32)).cuda()
    xd = to_dev(x, cfg.dtype)
    ws = m.store.workspace(1, k, steps)
    st = _status()
    y1 = torch.full((steps, d), 7.0, dtype=torch.float32, device="cuda")
    for s in range(steps):
        api.si_ffn_forward(m.store.handle, s % L, xd[s:s + 1], 1, idx[s].clone(), None, k, y1[s:s + 1], 0, ws, st)
    ys = torch.full((steps, d), 7.0, dtype=tdt, device="cuda")
    api.si_decode_stack_forward(m.store.handle, steps, None, xd, idx, None, k, ys, 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0, api.strerror(int(st.item()))
    for s in range(steps):
        ref = m.oracle_y(s % L, x[s], lists[s])
        assert_close(from_dev(y1[s]), ref, f"d={d} single step {s}")
        assert_close(from_dev(ys[s]), ref, f"d={d} stacked step {s}")

    # ---- several tokens with lists of their own: the union path (forced for 3 tokens, default for 40)
    for T, flags in ((3, api.SI_FLAG_UNION_PATH), (40, 0)):
        tl = wl.zipf_lists(cfg, 1, T, slot_of_rank=m.slot_of_rank[1])
        tx = wl.x_tokens(cfg, 1, T)
        wsT = m.store.workspace(T, k, 1)
        y = torch.full((T, d), 3.0, dtype=torch.float32, device="cuda")
        api.si_ffn_forward(m.store.handle, 1, to_dev(tx, cfg.dtype), T, torch.from_numpy(tl).cuda(), None, k, y, flags,
                           wsT, st)
        torch.cuda.synchronize()
        assert st.item() == 0, api.strerror(int(st.item()))
        for t in range(0, T, 1 if T <= 8 else 7):
            assert_close(from_dev(y[t]), m.oracle_y(1, tx[t], tl[t]), f"d={d} T={T} token {t}")

    # ---- 130 tokens on one shared list (two token tiles), residual added, 16-bit output
    T = 130
    shared = np.arange(k, dtype=np.int32)
    tx = wl.x_tokens(cfg, 0, T)
    wsT = m.store.workspace(T, k, 1)
    y = torch.full((T, d), 3.0, dtype=tdt, device="cuda")
    api.si_ffn_forward(m.store.handle, 0, to_dev(tx, cfg.dtype), T, torch.from_numpy(shared).cuda(), None, k, y,
                       api.SI_FLAG_SHARED_LIST | api.SI_FLAG_RESIDUAL, wsT, st)
    torch.cuda.synchronize()
    assert st.item() == 0, api.strerror(int(st.item()))
    for t in (0, 63, 128, 129):
        ref = m.oracle_y(0, tx[t], shared) + wl.bits_to_float64(tx[t], cfg.dtype)
        assert_close(from_dev(y[t]), ref, f"d={d} shared list token {t}")
