"""GPU parity: loader and batch-1 selective decode through the C ABI vs the float64 oracle."""
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


@pytest.fixture(scope="module")
def c1(api):
    return LoadedModel(wl.CONFIGS["c1"])


def _tiny_cfg(dtype="bf16", d_model=64, d_ff=96, loaded_pct=50):
    return wl.Config("tiny", 90, d_model, d_ff, 2, dtype, loaded_pct, 25, 4, loaded_rule="perm")


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


# ------------------------------------------------------------------ loader (a1)

@pytest.mark.parametrize("cfg_name", ["c1", "tiny"])
def test_loader_records_are_exact_slices(api, c1, cfg_name):
    m = c1 if cfg_name == "c1" else LoadedModel(_tiny_cfg())
    cfg = m.cfg
    for l in range(m.L):
        rec = m.store.records(l).view(torch.int16).cpu().numpy().view(np.uint16)   # [n_ld, 3, d]
        wg, wu, wd = m.host[l]
        ids = m.ids[l]
        assert np.array_equal(rec[:, 0, :], wg[ids])
        assert np.array_equal(rec[:, 1, :], wu[ids])
        assert np.array_equal(rec[:, 2, :], wd[:, ids].T)
        s2g, g2s = (t.cpu().numpy() for t in m.store.slot_maps(l))
        assert np.array_equal(s2g, ids)
        assert np.array_equal(g2s[ids], np.arange(len(ids)))
        assert np.all(g2s[np.setdiff1d(np.arange(cfg.d_ff), ids)] == -1)


def test_loader_rejects_bad_neuron_files(api):
    cfg = _tiny_cfg()
    store = api.NeuronStore(1, cfg.d_model, cfg.d_ff, [4], cfg.dtype)
    w = torch.zeros(cfg.d_ff, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    wd = torch.zeros(cfg.d_model, cfg.d_ff, dtype=torch.bfloat16, device="cuda")
    for ids, code in (([0, 1, 2, 96], api.SI_ERR_OUT_OF_RANGE), ([0, 1, 1, 2], api.SI_ERR_DUPLICATE),
                      ([0, 1, 2], api.SI_ERR_INVALID_ARG), ([-1, 1, 2, 3], api.SI_ERR_OUT_OF_RANGE)):
        with pytest.raises(api.SelectInferError) as e:
            store.load(0, w, w, wd, ids, 0)
        assert e.value.status == code
    with pytest.raises(api.SelectInferError):
        store.load(1, w, w, wd, [0, 1, 2, 3], 0)


# ------------------------------------------------------------------ decode (a2)

@pytest.mark.parametrize("flags_name", ["persistent", "simple"])
@pytest.mark.parametrize("y_f32", [True, False])
def test_c1_decode_matches_oracle(api, c1, flags_name, y_f32):
    cfg = c1.cfg
    flags = api.SI_FLAG_SIMPLE_KERNELS if flags_name == "simple" else 0
    lists = wl.zipf_lists(cfg, 0, cfg.tokens, slot_of_rank=c1.slot_of_rank[0])
    x = wl.x_tokens(cfg, 0, cfg.tokens)
    ws = c1.store.workspace(1, cfg.k_active, cfg.tokens)
    xd, idx = to_dev(x, cfg.dtype), torch.from_numpy(lists).cuda()
    ydt = torch.float32 if y_f32 else xd.dtype
    st = _status()
    # one call per token ...
    y = torch.empty(cfg.tokens, cfg.d_model, dtype=ydt, device="cuda")
    for t in range(cfg.tokens):
        api.si_ffn_forward(c1.store.handle, 0, xd[t], 1, idx[t], None, cfg.k_active, y[t], flags, ws, st)
    # ... and all tokens as one stack call
    y2 = torch.empty_like(y)
    api.si_decode_stack_forward(c1.store.handle, cfg.tokens, [0] * cfg.tokens, xd, idx, None, cfg.k_active, y2,
                                flags, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for t in range(cfg.tokens):
        ref = c1.oracle_y(0, x[t], lists[t])
        assert_close(from_dev(y[t]), ref, f"token {t} single")
        assert_close(from_dev(y2[t]), ref, f"token {t} stack")


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("flags_name", ["persistent", "simple"])
def test_tiny_degenerate_lists(api, dtype, flags_name):
    """k in {0, 1, 2, n_loaded}; shuffled list; residual; against the oracle."""
    cfg = _tiny_cfg(dtype)
    m = LoadedModel(cfg)
    flags0 = api.SI_FLAG_SIMPLE_KERNELS if flags_name == "simple" else 0
    n = cfg.n_loaded
    x = wl.x_tokens(cfg, 1, 1)[0]
    xd = to_dev(x, dtype)
    ws = m.store.workspace(1, n, 4)
    g = np.random.default_rng(5)
    for k in (0, 1, 2, n):
        slots = np.sort(g.permutation(n)[:k]).astype(np.int32)
        idx = torch.from_numpy(slots if k else np.zeros(4, np.int32)).cuda()
        for residual in (False, True):
            y = torch.full((cfg.d_model,), 7.0, dtype=torch.float32, device="cuda")
            st = _status()
            api.si_ffn_forward(m.store.handle, 1, xd, 1, idx, None, k, y,
                               flags0 | (api.SI_FLAG_RESIDUAL if residual else 0), ws, st)
            torch.cuda.synchronize()
            assert st.item() == 0
            ref = m.oracle_y(1, x, slots)
            if residual:
                ref = ref + wl.bits_to_float64(x, dtype)
            if k == 0 and not residual:
                assert np.array_equal(from_dev(y), np.zeros(cfg.d_model))
            else:
                assert_close(from_dev(y), ref, f"k={k} residual={residual}")
    # list order does not matter: bit-identical output for a shuffled list
    slots = np.sort(g.permutation(n)[:9]).astype(np.int32)
    ya = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    yb = torch.empty_like(ya)
    api.si_ffn_forward(m.store.handle, 0, xd, 1, torch.from_numpy(slots).cuda(), None, 9, ya, flags0, ws, None)
    shuffled = slots[g.permutation(9)].copy()
    api.si_ffn_forward(m.store.handle, 0, xd, 1, torch.from_numpy(shuffled).cuda(), None, 9, yb, flags0, ws, None)
    torch.cuda.synchronize()
    assert_close(from_dev(yb), m.oracle_y(0, x, slots), "shuffled")
    assert_close(from_dev(ya), m.oracle_y(0, x, slots), "sorted")


@pytest.mark.parametrize("flags_name", ["persistent", "simple"])
def test_ragged_csr_lists_over_a_stack(api, flags_name):
    """CSR lists of different lengths (one empty) over a 2-layer stack in one call."""
    cfg = _tiny_cfg("bf16", d_model=256, d_ff=400, loaded_pct=60)
    m = LoadedModel(cfg)
    flags = api.SI_FLAG_SIMPLE_KERNELS if flags_name == "simple" else 0
    n = cfg.n_loaded
    g = np.random.default_rng(6)
    lens = [5, 0, n, 37, 1, 150]
    layers = [0, 1, 1, 0, 1, 0]
    lists = [np.sort(g.permutation(n)[:k]).astype(np.int32) for k in lens]
    offsets = np.zeros(len(lens) + 1, np.int32); offsets[1:] = np.cumsum(lens)
    flat = np.concatenate(lists).astype(np.int32)
    x = np.stack([wl.x_tokens(cfg, layers[s], 1, first_token=s)[0] for s in range(len(lens))])
    xd = to_dev(x, cfg.dtype)
    y = torch.empty(len(lens), cfg.d_model, dtype=torch.float32, device="cuda")
    ws = m.store.workspace(1, n, len(lens))
    st = _status()
    api.si_decode_stack_forward(m.store.handle, len(lens), layers, xd, torch.from_numpy(flat).cuda(),
                                torch.from_numpy(offsets).cuda(), n, y, flags | api.SI_FLAG_CHECK, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for s in range(len(lens)):
        ref = m.oracle_y(layers[s], x[s], lists[s])
        if lens[s] == 0:
            assert np.array_equal(from_dev(y[s]), np.zeros(cfg.d_model))
        else:
            assert_close(from_dev(y[s]), ref, f"step {s}")


@pytest.mark.parametrize("flags_name", ["persistent", "simple"])
def test_stack_with_one_list_per_layer(api, flags_name):
    """The paper's decode: the set chosen for a layer stays fixed for the prompt, so the stack call takes
    one list per layer.  Results equal the same call with the list repeated for every step, bit for bit."""
    cfg = _tiny_cfg("bf16", d_model=256, d_ff=400, loaded_pct=60)
    m = LoadedModel(cfg)
    base = api.SI_FLAG_SIMPLE_KERNELS if flags_name == "simple" else 0
    L, tokens, n = m.L, 5, cfg.n_loaded
    k = n // 3
    g = np.random.default_rng(12)
    lists = np.stack([np.sort(g.permutation(n)[:k]).astype(np.int32) for _ in range(L)])     # [L, k]
    n_steps = tokens * L
    x = np.stack([wl.x_tokens(cfg, s % L, 1, first_token=s // L)[0] for s in range(n_steps)])
    xd = to_dev(x, cfg.dtype)
    ws = m.store.workspace(1, k, n_steps)
    y1 = torch.empty(n_steps, cfg.d_model, dtype=torch.float32, device="cuda")
    y2 = torch.empty_like(y1)
    st = _status()
    api.si_decode_stack_forward(m.store.handle, n_steps, None, xd, torch.from_numpy(lists).cuda(), None, k, y1,
                                base | api.SI_FLAG_LIST_PER_LAYER | api.SI_FLAG_CHECK, ws, st)
    per_step = np.stack([lists[s % L] for s in range(n_steps)])
    api.si_decode_stack_forward(m.store.handle, n_steps, None, xd, torch.from_numpy(per_step).cuda(), None, k, y2,
                                base, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert torch.equal(y1, y2)
    for s in (0, 1, L, n_steps - 1):
        assert_close(from_dev(y1[s]), m.oracle_y(s % L, x[s], lists[s % L]), f"step {s}")
    # custom layer order
    order = [1, 0, 1, 1, 0]
    y3 = torch.empty(len(order), cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_decode_stack_forward(m.store.handle, len(order), order, xd[: len(order)], torch.from_numpy(lists).cuda(),
                                None, k, y3, base | api.SI_FLAG_LIST_PER_LAYER, ws, st)
    torch.cuda.synchronize()
    for s, l in enumerate(order):
        assert_close(from_dev(y3[s]), m.oracle_y(l, x[s], lists[l]), f"ordered step {s}")


def test_7b_shaped_two_layers_stack_and_determinism(api):
    """Llama-2-7B FFN shape (d_model 4096, d_ff 11008, bf16), 2 layers x 3 tokens: spans many
    SMs, several ring passes and a ragged tail of records per SM."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=2)
    tokens, L, k = 3, 2, cfg.k_active
    x = np.stack([wl.x_tokens(cfg, l, tokens) for l in range(L)], axis=1)          # [tokens, L, d]
    lists = np.stack([wl.zipf_lists(cfg, l, tokens) for l in range(L)], axis=1)     # [tokens, L, k]
    xd = to_dev(x.reshape(tokens * L, -1), cfg.dtype)
    idx = torch.from_numpy(lists.reshape(tokens * L, k)).cuda()
    ws = m.store.workspace(1, k, tokens * L)
    outs = []
    for flags in (0, 0, api.SI_FLAG_SIMPLE_KERNELS):
        y = torch.empty(tokens * L, cfg.d_model, dtype=torch.float32, device="cuda")
        st = _status()
        api.si_decode_stack_forward(m.store.handle, tokens * L, None, xd, idx, None, k, y, flags, ws, st)
        torch.cuda.synchronize()
        assert st.item() == 0
        outs.append(y.cpu())
    assert torch.equal(outs[0], outs[1]), "persistent kernel is not run-to-run bit-stable"
    for s in range(tokens * L):
        t, l = divmod(s, L)
        ref = m.oracle_y(l, x[t, l], lists[t, l])
        assert_close(outs[0][s].double().numpy(), ref, f"persistent step {s}")
        assert_close(outs[2][s].double().numpy(), ref, f"simple step {s}")
    # bf16 output
    yb = torch.empty(tokens * L, cfg.d_model, dtype=torch.bfloat16, device="cuda")
    api.si_decode_stack_forward(m.store.handle, tokens * L, None, xd, idx, None, k, yb, 0, ws, None)
    torch.cuda.synchronize()
    assert_close(from_dev(yb[3]), m.oracle_y(1, x[1, 1], lists[1, 1]), "bf16 out")


def test_7b_shaped_step_groups(api):
    """The persistent kernel with its SMs split into 1, 2 and 4 step groups (one by default, up to
    four with SI_FLAG_STEPS_ANY_ORDER for launches of 8 steps or more): 13 steps, so the groups get 4, 3, 3 and 3 steps; lists of equal
    length, ragged lists with offsets (an empty one among them) and one list per layer; residual."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=2)
    steps, L, k, n = 13, 2, cfg.k_active, cfg.n_loaded
    g = np.random.default_rng(77)
    x = np.stack([wl.x_tokens(cfg, s % L, 1, first_token=s)[0] for s in range(steps)])
    xd = to_dev(x, cfg.dtype)
    fixed = np.stack([wl.zipf_lists(cfg, s % L, 1, first_token=s)[0] for s in range(steps)])
    lens = [int(v) for v in g.integers(1, 2 * k, size=steps)]
    lens[4] = 0
    ragged = [np.sort(g.permutation(n)[:c]).astype(np.int32) for c in lens]
    off = np.zeros(steps + 1, dtype=np.int32)
    off[1:] = np.cumsum(lens)
    per_layer = np.stack([wl.zipf_lists(cfg, l, 1)[0] for l in range(L)])
    ws = m.store.workspace(1, max(max(lens), k), steps)
    cases = [
        ("fixed", torch.from_numpy(fixed).cuda(), None, k, 0, lambda s: fixed[s]),
        ("offsets", torch.from_numpy(np.concatenate(ragged + [np.zeros(4, np.int32)])).cuda(), torch.from_numpy(off).cuda(),
         max(lens), api.SI_FLAG_RESIDUAL, lambda s: ragged[s]),
        ("per layer", torch.from_numpy(per_layer).cuda(), None, k, api.SI_FLAG_LIST_PER_LAYER, lambda s: per_layer[s % L]),
    ]
    for name, idx, offsets, kk, flags, list_of in cases:
        refs = None
        for ng in (1, 2, 4, 0):       # 0: the library's own choice under SI_FLAG_STEPS_ANY_ORDER
            runs = []
            for _ in range(2):
                y = torch.full((steps, cfg.d_model), 9.0, dtype=torch.float32, device="cuda")
                st = _status()
                # (the per-call option fixes the group count; the flag is what a caller would pass for more than one)
                api.si_debug_decode_stack_forward(m.store.handle, steps, None, xd, idx, offsets, kk, y,
                                                  flags | (api.SI_FLAG_STEPS_ANY_ORDER if ng != 1 else 0), ws, st,
                                                  step_groups=ng)
                torch.cuda.synchronize()
                assert st.item() == 0, (name, ng, api.strerror(int(st.item())))
                runs.append(y.cpu())
            assert torch.equal(runs[0], runs[1]), f"{name}: {ng} groups not run-to-run bit-stable"
            if refs is None:
                refs = []
                for s in range(steps):
                    ref = m.oracle_y(s % L, x[s], list_of(s))
                    if flags & api.SI_FLAG_RESIDUAL:
                        ref = ref + wl.bits_to_float64(x[s], cfg.dtype)
                    refs.append(ref)
            for s in range(steps):
                assert_close_f32(runs[0][s].double().numpy(), refs[s], f"{name}, {ng} groups, step {s}")


def test_check_flag_reports_bad_lists_without_faulting(api):
    cfg = _tiny_cfg()
    m = LoadedModel(cfg)
    n = cfg.n_loaded
    xd = to_dev(wl.x_tokens(cfg, 0, 1)[0], cfg.dtype)
    y = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    ws = m.store.workspace(1, n, 1)
    for bad, code in (([0, 3, 3, 5], api.SI_ERR_DUPLICATE), ([0, 3, n, 5], api.SI_ERR_OUT_OF_RANGE),
                      ([0, -2, 4, 5], api.SI_ERR_OUT_OF_RANGE)):
        for flags in (api.SI_FLAG_CHECK, api.SI_FLAG_CHECK | api.SI_FLAG_SIMPLE_KERNELS):
            st = _status()
            api.si_ffn_forward(m.store.handle, 0, xd, 1, torch.tensor(bad, dtype=torch.int32, device="cuda"),
                               None, 4, y, flags, ws, st)
            torch.cuda.synchronize()
            assert st.item() == code
    # out-of-range is also caught (and skipped) without the check flag
    st = _status()
    api.si_ffn_forward(m.store.handle, 0, xd, 1, torch.tensor([0, 3, n + 7, 5], dtype=torch.int32, device="cuda"),
                       None, 4, y, 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == api.SI_ERR_OUT_OF_RANGE
    ref = m.oracle_y(0, wl.x_tokens(cfg, 0, 1)[0], [0, 3, 5])
    assert_close(from_dev(y), ref, "bad entry skipped")


def test_host_side_argument_errors(api, c1):
    cfg = c1.cfg
    xd = to_dev(wl.x_tokens(cfg, 0, 1)[0], cfg.dtype)
    y = torch.empty(cfg.d_model, dtype=torch.float32, device="cuda")
    idx = torch.zeros(8, dtype=torch.int32, device="cuda")
    ws = c1.store.workspace(1, cfg.k_active, 1)

    def status_of(fn):
        with pytest.raises(api.SelectInferError) as e:
            fn()
        return e.value.status

    h = c1.store.handle
    assert status_of(lambda: api.si_ffn_forward(h, 3, xd, 1, idx, None, 4, y, 0, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_ffn_forward(h, 0, xd, 0, idx, None, 4, y, 0, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_ffn_forward(h, 0, xd, 1, idx, None, cfg.n_loaded + 1, y, 0, ws)) == api.SI_ERR_OUT_OF_RANGE
    assert status_of(lambda: api.si_ffn_forward(h, 0, xd, 1, idx, None, 4, y, 0, ws[:256])) == api.SI_ERR_NOMEM
    assert status_of(lambda: api.si_ffn_forward(h, 0, xd[1:], 1, idx, None, 4, y[1:], 0, ws)) == api.SI_ERR_ALIGNMENT
    yh = torch.empty(cfg.d_model, dtype=torch.bfloat16, device="cuda")     # store is fp16
    assert status_of(lambda: api.si_ffn_forward(h, 0, xd, 1, idx, None, 4, yh, 0, ws)) == api.SI_ERR_INVALID_ARG


def test_unloaded_layer_is_refused_before_anything_runs(api):
    """A layer that was never loaded is refused on the host before anything is enqueued (single call, selector
    call, stack call)."""
    cfg = _tiny_cfg()
    store = api.NeuronStore(2, cfg.d_model, cfg.d_ff, [cfg.n_loaded] * 2, cfg.dtype)
    wg, wu, wd = wl.layer_weights(cfg, 0)
    ids, _ = wl.loaded_ids(cfg, 0)
    store.load(0, to_dev(wg, cfg.dtype), to_dev(wu, cfg.dtype), to_dev(wd, cfg.dtype), ids, cfg.n_base)   # layer 1 stays unloaded
    n = cfg.n_loaded
    xd = to_dev(wl.x_tokens(cfg, 0, 4), cfg.dtype)
    y = torch.full((4, cfg.d_model), 5.0, dtype=torch.float32, device="cuda")
    idx = torch.zeros(16, dtype=torch.int32, device="cuda")
    scores = torch.zeros(n, dtype=torch.float32, device="cuda")
    ws = store.workspace(1, n, 4)
    st = _status()

    def status_of(fn):
        with pytest.raises(api.SelectInferError) as e:
            fn()
        return e.value.status

    assert status_of(lambda: api.si_ffn_forward(store.handle, 1, xd[0], 1, idx, None, 4, y[0], 0, ws, st)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_layer_forward(store.handle, 1, xd[0], 1, scores, 4, None, None, y[0], 0, ws, st)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_decode_stack_forward(store.handle, 4, [0, 0, 1, 0], xd, idx, None, 4, y, api.SI_FLAG_CHECK, ws, st)) \
        == api.SI_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert st.item() == 0 and bool((y == 5.0).all())                  # nothing ran
    store.close()
