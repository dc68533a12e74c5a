"""GPU parity of the decode with a static prefix (the static neurons are the first slots of the store and are
streamed without list entries; the lists hold the dynamic neurons only) against the float64 oracle and,
bit for bit, against the same steps given as explicit lists."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, assert_close_f32, from_dev, to_dev

pytestmark = pytest.mark.gpu

EPS = 1e-5


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _dynamic_lists(seed, n_lists, n_static, n_loaded, k_dyn):
    g = np.random.default_rng(seed)
    return np.stack([np.sort(n_static + g.permutation(n_loaded - n_static)[:k_dyn]).astype(np.int32) for _ in range(n_lists)])


def test_c1_prefix_independent_steps(api):
    """Sixteen independent steps on the config-1 model: 100 static slots plus 60 listed ones per step, fp32 out,
    against the oracle on the union and bit for bit against the explicit lists [0..99] + listed."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    n_steps, n_static, k_dyn = 16, 100, 60
    dyn = _dynamic_lists(3, n_steps, n_static, cfg.n_loaded, k_dyn)
    full = np.concatenate([np.tile(np.arange(n_static, dtype=np.int32), (n_steps, 1)), dyn], axis=1)
    x = wl.x_tokens(cfg, 0, n_steps, first_token=70)
    xd = to_dev(x, cfg.dtype)
    ws = m.store.workspace(1, n_static + k_dyn, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    for flags in (0, api.SI_FLAG_RESIDUAL | api.SI_FLAG_CHECK):
        y = torch.empty(n_steps, cfg.d_model, dtype=torch.float32, device="cuda")
        api.si_decode_prefix_forward(m.store.handle, n_steps, [0] * n_steps, n_static, 0, xd, torch.from_numpy(dyn).cuda(), None, k_dyn,
                                     y, None, 0.0, flags, ws, st)
        y_full = torch.empty_like(y)
        api.si_decode_stack_forward(m.store.handle, n_steps, [0] * n_steps, xd, torch.from_numpy(full).cuda(), None, n_static + k_dyn,
                                    y_full, flags, ws, st)
        torch.cuda.synchronize()
        assert st.item() == 0, api.strerror(int(st.item()))
        assert torch.equal(y, y_full)
        for s in range(n_steps):
            ref = m.oracle_y(0, x[s], full[s])
            if flags & api.SI_FLAG_RESIDUAL:
                ref = ref + wl.bits_to_float64(x[s], cfg.dtype)
            assert_close_f32(from_dev(y[s]), ref, f"step {s}")
    # static neurons only: no list at all
    y = torch.empty(n_steps, cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_decode_prefix_forward(m.store.handle, n_steps, [0] * n_steps, n_static, 0, xd, None, None, 0, y, None, 0.0, 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert_close_f32(from_dev(y[5]), m.oracle_y(0, x[5], np.arange(n_static)), "static neurons only")
    # a listed slot inside the prefix repeats a static neuron: reported under the check flag
    bad = dyn.copy()
    bad[3, 0] = 7
    api.si_decode_prefix_forward(m.store.handle, n_steps, [0] * n_steps, n_static, 0, xd, torch.from_numpy(bad).cuda(), None, k_dyn,
                                 y, None, 0.0, api.SI_FLAG_CHECK, ws, st)
    torch.cuda.synchronize()
    assert st.item() == api.SI_ERR_DUPLICATE
    with pytest.raises(api.SelectInferError) as e:
        api.si_decode_prefix_forward(m.store.handle, n_steps, [0] * n_steps, cfg.n_loaded - 10, 0, xd, torch.from_numpy(dyn).cuda(), None,
                                     k_dyn, y, None, 0.0, 0, ws, st)
    assert e.value.status == api.SI_ERR_OUT_OF_RANGE


@pytest.mark.parametrize("form", [1, 2])
def test_c1_prefix_chained_equals_explicit_lists(api, form):
    """Chains of four steps with pre-norm and residual: the prefix call and the call with explicit lists give the
    same bits in either form of the chained kernel, and every step matches the oracle fed with the device's input."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    n_steps, chain_len, n_static, k_dyn = 12, 4, 100, 60
    dyn = _dynamic_lists(4, n_steps, n_static, cfg.n_loaded, k_dyn)
    full = np.concatenate([np.tile(np.arange(n_static, dtype=np.int32), (n_steps, 1)), dyn], axis=1)
    heads = wl.x_tokens(cfg, 0, n_steps // chain_len, first_token=90)
    hd = to_dev(heads, cfg.dtype)
    ws = m.store.workspace(1, n_static + k_dyn, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    flags = api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL
    y = torch.empty(n_steps, cfg.d_model, dtype=torch.float16, device="cuda")
    xn = torch.empty_like(y)
    api.si_decode_prefix_forward(m.store.handle, n_steps, [0] * n_steps, n_static, chain_len, hd, torch.from_numpy(dyn).cuda(), None, k_dyn,
                                 y, xn, EPS, flags, ws, st)
    y_full = torch.empty_like(y)
    api.si_debug_decode_chain_forward(m.store.handle, n_steps, [0] * n_steps, chain_len, hd, torch.from_numpy(full).cuda(), None,
                                      n_static + k_dyn, y_full, None, EPS, flags, ws, st, chain_form=form)
    torch.cuda.synchronize()
    assert st.item() == 0, api.strerror(int(st.item()))
    if form == 2:                     # the prefix call takes the library's choice of form, which here is the split one
        assert torch.equal(y, y_full)
    yb = y.view(torch.int16).cpu().numpy().view(np.uint16)
    xnb = xn.view(torch.int16).cpu().numpy().view(np.uint16)
    for s in range(n_steps):
        in_bits = heads[s // chain_len] if s % chain_len == 0 else yb[s - 1]
        ref = m.oracle_y(0, xnb[s], full[s]) + so.widen_bits(in_bits, cfg.dtype)
        assert_close(so.widen_bits(yb[s], cfg.dtype), ref, f"step {s}")
        assert_close(from_dev(y_full[s]), ref, f"step {s}, explicit lists, form {form}")


def test_7b_prefix_table1_counts(api):
    """7B-shaped layers with the paper's default split (Table 1): the static neurons are 30 % of d_ff (3302 slots, the
    store's first), the dynamic ones 10 % (1101 listed slots), 4403 computed of 7705 loaded.  Independent steps and
    chains over two layers, sampled steps against the oracle."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=2)
    L, tokens = 2, 5
    n_steps = L * tokens
    n_static, k_dyn = wl.count_pct(30, cfg.d_ff), wl.count_pct(10, cfg.d_ff)
    assert (n_static, k_dyn, cfg.n_loaded) == (3302, 1100, 7705)
    dyn = _dynamic_lists(5, n_steps, n_static, cfg.n_loaded, k_dyn)
    full = np.concatenate([np.tile(np.arange(n_static, dtype=np.int32), (n_steps, 1)), dyn], axis=1)
    x = np.stack([wl.x_tokens(cfg, s % L, 1, first_token=400 + s)[0] for s in range(n_steps)])
    xd = to_dev(x, cfg.dtype)
    ws = m.store.workspace(1, n_static + k_dyn, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(n_steps, cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_decode_prefix_forward(m.store.handle, n_steps, None, n_static, 0, xd, torch.from_numpy(dyn).cuda(), None, k_dyn, y, None, 0.0,
                                 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for s in (0, 3, n_steps - 1):
        assert_close_f32(from_dev(y[s]), m.oracle_y(s % L, x[s], full[s]), f"independent step {s}")
    # chains through both layers
    heads = x[::L].copy()
    yc = torch.empty(n_steps, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    xn = torch.empty_like(yc)
    flags = api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL
    api.si_decode_prefix_forward(m.store.handle, n_steps, None, n_static, L, to_dev(heads, cfg.dtype), torch.from_numpy(dyn).cuda(), None,
                                 k_dyn, yc, xn, EPS, flags, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    yb = yc.view(torch.int16).cpu().numpy().view(np.uint16)
    xnb = xn.view(torch.int16).cpu().numpy().view(np.uint16)
    for s in (0, 1, 6, 9):
        in_bits = heads[s // L] if s % L == 0 else yb[s - 1]
        ref = m.oracle_y(s % L, xnb[s], full[s]) + so.widen_bits(in_bits, cfg.dtype)
        assert_close(so.widen_bits(yb[s], cfg.dtype), ref, f"chained step {s}")
