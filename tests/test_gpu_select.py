"""GPU parity: runtime selector (bit-exact vs the oracle) and the layer wrapper."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _run_select(api, scores, mode, k=0, tau=0.0, flags=0, cap=None):
    s = torch.from_numpy(np.asarray(scores, dtype=np.float32)).cuda()
    n = s.numel()
    cap = n if cap is None else cap
    out = torch.full((max(cap, 4),), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    ws = torch.zeros(max(api.si_select_workspace_bytes(n), 256), dtype=torch.uint8, device="cuda")
    api._check(api.lib().si_select(api._dp(s), n, mode, k, tau, flags, api._dp(out), cap, api._dp(cnt), api._dp(ws),
                                   ws.numel(), api._stream()), "si_select")
    torch.cuda.synchronize()
    c = int(cnt[0].item())
    return out[:min(c, cap)].cpu().numpy(), c


ADVERSARIAL = [
    [0.5, -1.0, 3.0, 3.0, 0.0, -0.0, 2.0],
    [1.0] * 9,
    [float("nan"), 1.0, float("-inf"), float("inf"), float("nan"), 0.0, -0.0],
    [-3.0, -2.0, -2.0, -2.0, -1.0, -2.0, -5.0],
    [0.0, -0.0, 0.0, -0.0, 0.0, -0.0, 1e-45, -1e-45],
]


@pytest.mark.parametrize("scores", ADVERSARIAL)
def test_topk_adversarial_ties_bit_exact(api, scores):
    for use_abs in (False, True):
        for k in range(len(scores) + 1):
            got, c = _run_select(api, scores, api.SI_SELECT_TOPK, k=k, flags=api.SI_FLAG_SCORE_ABS if use_abs else 0)
            want = so.select_topk(scores, k, use_abs=use_abs)
            assert c == k and np.array_equal(got, want), (scores, k, use_abs, got, want)


@pytest.mark.parametrize("n,k", [(1, 1), (33, 7), (1000, 400), (4300, 215), (7705, 1541), (14336, 7168),
                                 (14336, 0), (14336, 14336), (16385, 1), (20000, 19999), (28672, 5734),
                                 (40000, 777), (50000, 12345), (70000, 3000)])
def test_topk_random_and_tied_scores(api, n, k):
    g = np.random.default_rng(n + k)
    for tied in (False, True):
        s = g.standard_normal(n).astype(np.float32)
        if tied:
            s = np.round(s, 1)           # blocks of equal values straddle the k boundary
        got, c = _run_select(api, s, api.SI_SELECT_TOPK, k=k)
        want = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k]).astype(np.int32)
        assert c == k and np.array_equal(got, want)
        if n <= 5000:
            assert np.array_equal(got, so.select_topk(s, k))


def test_threshold_mode_and_capacity(api):
    g = np.random.default_rng(3)
    s = g.standard_normal(5000).astype(np.float32)
    s[17] = np.nan
    for tau, use_abs in ((0.5, False), (-10.0, False), (10.0, False), (1.0, True)):
        got, c = _run_select(api, s, api.SI_SELECT_THRESHOLD, tau=tau, flags=api.SI_FLAG_SCORE_ABS if use_abs else 0)
        want = so.select_threshold(s, tau, use_abs=use_abs)
        assert c == len(want) and np.array_equal(got, want)
    want = so.select_threshold(s, 0.0)
    got, c = _run_select(api, s, api.SI_SELECT_THRESHOLD, tau=0.0, cap=100)
    assert c == len(want) and np.array_equal(got, want[:100])      # full count, truncated list
    with pytest.raises(api.SelectInferError) as e:
        _run_select(api, s, api.SI_SELECT_TOPK, k=200, cap=100)
    assert e.value.status == api.SI_ERR_NOMEM
    with pytest.raises(api.SelectInferError):
        _run_select(api, s, api.SI_SELECT_TOPK, k=5001)


def test_c5_scores_select_all_cells(api):
    """Config-5 selector inputs: N(0,1) scores over the loaded slots, k per cell, signed ranking."""
    cfg0 = wl.CONFIGS["c5"]
    for lp in wl.C5_LOADED:
        cfg = cfg0.with_(loaded_pct=lp)
        sc = wl.scores(cfg, 3, 2)
        for ap in wl.C5_ACTIVE:
            k = wl.count_pct(ap, cfg.n_loaded)
            for t in range(2):
                got, c = _run_select(api, sc[t], api.SI_SELECT_TOPK, k=k)
                want = np.sort(np.argsort(-sc[t].astype(np.float64), kind="stable")[:k]).astype(np.int32)
                assert c == k and np.array_equal(got, want)
        assert np.array_equal(_run_select(api, sc[0][:3000], api.SI_SELECT_TOPK, k=300)[0],
                              so.select_topk(sc[0][:3000], 300))


def test_layer_forward_selects_then_computes(api):
    """si_layer_forward with scores == oracle top-k followed by the oracle FFN on that list."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    n, k = cfg.n_loaded, cfg.k_active
    sc = wl.scores(cfg, 0, 2)
    x = wl.x_tokens(cfg, 0, 2)
    ws = m.store.workspace(1, k, 1)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    for t in range(2):
        y = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
        api.si_layer_forward(m.store.handle, 0, to_dev(x[t], cfg.dtype), 1, torch.from_numpy(sc[t]).cuda(), k,
                             None, None, y, api.SI_FLAG_RESIDUAL, ws, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        slots = so.select_topk(sc[t], k)
        ref = m.oracle_y(0, x[t], slots) + wl.bits_to_float64(x[t], cfg.dtype)
        assert_close(from_dev(y), ref, f"token {t}")
    # without scores it is si_ffn_forward
    lists = wl.zipf_lists(cfg, 0, 1, slot_of_rank=m.slot_of_rank[0])
    y = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_layer_forward(m.store.handle, 0, to_dev(x[0], cfg.dtype), 1, None, k, torch.from_numpy(lists[0]).cuda(),
                         None, y, 0, ws, st)
    torch.cuda.synchronize()
    assert_close(from_dev(y), m.oracle_y(0, x[0], lists[0]), "explicit list")
