"""GPU parity at the benchmark configurations' full sizes, on sampled outputs the oracle can
compute one by one, in the launch configuration bench.py times."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, assert_close_f32, from_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def test_c2_full_stack_one_launch_sampled(api):
    """Config 2 exactly as benched: 32 layers x 128 tokens = 4096 steps in one persistent launch.
    Sampled (token, layer) steps are checked against the oracle; every output must be finite."""
    cfg = wl.CONFIGS["c2"]
    keep = (0, 17, 31)
    m = LoadedModel(cfg, keep_layers=keep)
    L, d, k, tokens = cfg.n_layers, cfg.d_model, cfg.k_active, cfg.tokens
    x = np.empty((tokens, L, d), dtype=np.uint16)
    lists = np.empty((tokens, L, k), dtype=np.int32)
    for l in range(L):
        x[:, l] = wl.x_tokens(cfg, l, tokens)
        lists[:, l] = wl.zipf_lists(cfg, l, tokens)
    n_steps = tokens * L
    xd = to_dev(x.reshape(n_steps, d), cfg.dtype)
    idx = torch.from_numpy(lists.reshape(n_steps, k)).cuda()
    y = torch.empty(n_steps, d, dtype=torch.bfloat16, device="cuda")
    ws = m.store.workspace(1, k, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.si_decode_stack_forward(m.store.handle, n_steps, None, xd, idx, None, k, y, 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert bool(torch.isfinite(y.float()).all())
    for t in (0, 63, 127):
        for l in keep:
            ref = m.oracle_y(l, x[t, l], lists[t, l])
            assert_close(from_dev(y[t * L + l]), ref, f"token {t} layer {l}")
    # the last steps of the launch go through the flush of the trailing reduction
    assert_close(from_dev(y[n_steps - 1]), m.oracle_y(31, x[127, 31], lists[127, 31]), "last step")
    # second launch on the same workspace: bit-identical
    y2 = torch.empty_like(y)
    api.si_decode_stack_forward(m.store.handle, n_steps, None, xd, idx, None, k, y2, 0, ws, st)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)


@pytest.mark.parametrize("loaded_pct", wl.C5_LOADED)
def test_c5_all_cells_decode_and_selector(api, loaded_pct):
    """Config 5 (Llama-3-8B FFN shape), all sixteen cells (four active fractions per loaded fraction, one
    layer): Zipf lists through the decode kernel in the stack call bench.py times, and N(0,1) scores through
    si_layer_forward (selector + FFN) with bit-exact selection."""
    base = wl.CONFIGS["c5"].with_(loaded_pct=loaded_pct, n_layers=1)
    m = LoadedModel(base)
    d, n = base.d_model, base.n_loaded
    tokens = 2
    x = wl.x_tokens(base, 0, tokens)
    sc = wl.scores(base, 0, 1)[0]
    scd = torch.from_numpy(sc).cuda()
    sws = torch.zeros(max(api.si_select_workspace_bytes(n), 256), dtype=torch.uint8, device="cuda")
    for active_pct in wl.C5_ACTIVE:
        cfg = base.with_(active_pct=active_pct)
        k = cfg.k_active
        lists = wl.zipf_lists(cfg, 0, tokens)
        ws = m.store.workspace(1, k, tokens)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        y = torch.empty(tokens, d, dtype=torch.float32, device="cuda")
        api.si_decode_stack_forward(m.store.handle, tokens, [0] * tokens, to_dev(x, cfg.dtype),
                                    torch.from_numpy(lists).cuda(), None, k, y, 0, ws, st)
        # the persistent kernel as well (a stack call of two steps uses the per-step kernels)
        y8 = torch.empty(8, d, dtype=torch.float32, device="cuda")
        x8 = to_dev(np.tile(x, (4, 1)), cfg.dtype)
        l8 = torch.from_numpy(np.tile(lists, (4, 1))).cuda()
        ws8 = m.store.workspace(1, k, 8)
        api.si_decode_stack_forward(m.store.handle, 8, [0] * 8, x8, l8, None, k, y8, 0, ws8, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        for t in range(tokens):
            ref = m.oracle_y(0, x[t], lists[t])
            assert_close_f32(from_dev(y[t]), ref, f"cell {loaded_pct}/{active_pct} token {t}")
            assert_close_f32(from_dev(y8[6 + t]), ref, f"cell {loaded_pct}/{active_pct} token {t}, persistent kernel")
        # runtime selector on the cell's scores, then the FFN on the selected list
        sel_out = torch.empty(k, dtype=torch.int32, device="cuda")
        cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
        api.si_select(scd, api.SI_SELECT_TOPK, k, 0.0, 0, sel_out, cnt, sws)
        ysel = torch.empty(d, dtype=torch.float32, device="cuda")
        api.si_layer_forward(m.store.handle, 0, to_dev(x[0], cfg.dtype), 1, scd, k, None, None, ysel, 0, ws, st)
        torch.cuda.synchronize()
        want = np.sort(np.argsort(-sc.astype(np.float64), kind="stable")[:k]).astype(np.int32)
        assert int(cnt[0].item()) == k and np.array_equal(sel_out.cpu().numpy(), want)
        assert np.array_equal(want, so.select_topk(sc, k))
        assert_close_f32(from_dev(ysel), m.oracle_y(0, x[0], want), f"cell {loaded_pct}/{active_pct} selected list")


def test_c4_prefill_own_model_all_tokens_two_layers(api):
    """Config 4 on a model built from config 4's own seeds: all 512 tokens of two layers, one shared list =
    the first 40 % of the loaded slots, every token against the oracle."""
    cfg = wl.CONFIGS["c4"]
    m = LoadedModel(cfg, n_layers=2)
    T, k, d = cfg.tokens, cfg.k_active, cfg.d_model
    assert (T, k) == (512, 3082)
    shared = np.arange(k, dtype=np.int32)
    idx = torch.from_numpy(shared).cuda()
    ws = m.store.workspace(T, k, 1)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    for layer in range(2):
        x = wl.x_tokens(cfg, layer, T)
        y = torch.empty(T, d, dtype=torch.bfloat16, device="cuda")
        api.si_ffn_forward(m.store.handle, layer, to_dev(x, cfg.dtype), T, idx, None, k, y, api.SI_FLAG_SHARED_LIST, ws, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        wg, wu, wd = m.host[layer]
        ref = so.ffn_tokens(wg, wu, wd, x, [m.ids[layer][shared]] * T, dtype=cfg.dtype, threads=so.host_threads())
        yh = from_dev(y)
        for t in range(T):
            assert_close(yh[t], ref[t], f"layer {layer} token {t}")
