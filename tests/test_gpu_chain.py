"""GPU parity of the chained decode (every step reads the output of the step before it) against the
float64 oracle, and the time-out path of the device-side waits."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev

pytestmark = pytest.mark.gpu

EPS = 1e-5


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def _run_chain(api, m, n_steps, chain_len, heads, lists_dev, offsets_dev, k, flags, want_xn=False, layers=None, **opts):
    cfg = m.cfg
    tdt = api.torch_dtype(cfg.dtype)
    y = torch.full((n_steps, cfg.d_model), 5.0, dtype=tdt, device="cuda")
    xn = torch.zeros(n_steps, cfg.d_model, dtype=tdt, device="cuda") if want_xn else None
    ws = m.store.workspace(1, k, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    if opts:
        api.si_debug_decode_chain_forward(m.store.handle, n_steps, layers, chain_len, heads, lists_dev, offsets_dev, k, y, xn,
                                          EPS, flags, ws, st, **opts)
    else:
        api.si_decode_chain_forward(m.store.handle, n_steps, layers, chain_len, heads, lists_dev, offsets_dev, k, y, xn,
                                    EPS, flags, ws, st)
    torch.cuda.synchronize()
    return y, xn, int(st.item())


def _check_steps_fed_with_device_inputs(api, m, y, xn, heads_bits, lists, chain_len, flags, steps, layer_of):
    """Every checked step against the oracle's FFN of the input the device itself read for it (its own
    rounded output of the step before), so the comparison does not compound along the chain; the
    normalised row is checked against the oracle's normalisation of that same input."""
    cfg = m.cfg
    yb = _bits(y)
    xnb = _bits(xn) if xn is not None else None
    ulp = 2.0 ** -8 if cfg.dtype == "bf16" else 2.0 ** -11
    for s in steps:
        in_bits = heads_bits[s // chain_len] if s % chain_len == 0 else yb[s - 1]
        xin = so.widen_bits(in_bits, cfg.dtype)
        if flags & api.SI_FLAG_PRENORM:
            want = so.rmsnorm(xin, EPS)
            got = so.widen_bits(xnb[s], cfg.dtype)
            # fp32 sum of squares and reciprocal root, then one rounding to 16 bits: within one unit of the
            # 16-bit type of the float64 value (half a unit of rounding plus the fp32 scale's error)
            assert np.all(np.abs(got - want) <= ulp * np.abs(want) + 1e-30), f"normalised input, step {s}"
            fed = xnb[s]
        else:
            fed = in_bits
        ref = m.oracle_y(layer_of(s), fed, lists[s])
        if flags & api.SI_FLAG_RESIDUAL:
            ref = ref + xin
        assert_close(so.widen_bits(yb[s], cfg.dtype), ref, f"step {s}")


@pytest.mark.parametrize("form", [1, 2])
@pytest.mark.parametrize("flags_name", ["plain", "residual", "prenorm", "prenorm+residual"])
def test_c1_chains_match_the_oracle(api, flags_name, form):
    """Config-1 model (fp16, one layer used over and over): 6 chains of 3 steps plus a ragged tail of 2, every
    step checked; and the whole chain against the oracle's own chain (its own rounding between steps).  Both
    forms of the chained kernel: the SMs exchange partial output rows (1) or the activations (2)."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    flags = {"plain": 0, "residual": api.SI_FLAG_RESIDUAL, "prenorm": api.SI_FLAG_PRENORM,
             "prenorm+residual": api.SI_FLAG_PRENORM | api.SI_FLAG_RESIDUAL}[flags_name]
    chain_len, n_steps, k = 3, 20, cfg.k_active
    n_chains = (n_steps + chain_len - 1) // chain_len
    heads = wl.x_tokens(cfg, 0, n_chains, first_token=40)
    if flags == 0:
        # without residual or normalisation the scale of a chain falls by about its square per step (h is a
        # product of two projections of the input) and the third output would underflow fp16: start eight
        # times larger (an exact scaling of the fp16 inputs), which keeps all three steps in the normal range
        heads = so.round_bits(so.widen_bits(heads, cfg.dtype) * 8.0, cfg.dtype)
    lists = wl.zipf_lists(cfg, 0, n_steps, slot_of_rank=m.slot_of_rank[0], first_token=40)
    y, xn, st = _run_chain(api, m, n_steps, chain_len, to_dev(heads, cfg.dtype), torch.from_numpy(lists).cuda(), None, k,
                           flags, want_xn=True, layers=[0] * n_steps, chain_form=form)
    assert st == 0, api.strerror(st)
    _check_steps_fed_with_device_inputs(api, m, y, xn if flags & api.SI_FLAG_PRENORM else None, heads, lists, chain_len,
                                        flags, range(n_steps), lambda s: 0)
    # the oracle's own chains, nothing taken from the device: rounding differences between the two sides
    # can flip a 16-bit value here and there, which three steps do not amplify beyond the tolerance
    for c in range(n_chains):
        s0, s1 = c * chain_len, min(n_steps, (c + 1) * chain_len)
        out, _, _ = so.ffn_chain({0: m.host[0]}, [0] * (s1 - s0), {0: m.ids[0]}, lists[s0:s1], heads[c], cfg.dtype,
                                 residual=bool(flags & api.SI_FLAG_RESIDUAL), prenorm=bool(flags & api.SI_FLAG_PRENORM),
                                 eps=EPS, threads=so.host_threads())
        for s in range(s0, s1):
            assert_close(from_dev(y[s]), so.widen_bits(out[s - s0], cfg.dtype), f"chain {c} step {s} (oracle's own chain)")
    # run-to-run bit stability
    y2, _, st = _run_chain(api, m, n_steps, chain_len, to_dev(heads, cfg.dtype), torch.from_numpy(lists).cuda(), None, k,
                           flags, layers=[0] * n_steps, chain_form=form)
    assert st == 0 and torch.equal(y, y2)


@pytest.mark.parametrize("form", [1, 2])
def test_7b_two_layers_eight_tokens_chained(api, form):
    """Config-2 shape: 8 tokens, each a chain through 2 layers; fixed lists, ragged lists with offsets (one
    of them empty) and one list per layer; plain, residual and pre-norm chains."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=2)
    L, tokens, k, n = 2, 8, cfg.k_active, cfg.n_loaded
    n_steps = L * tokens
    heads = wl.x_tokens(cfg, 0, tokens, first_token=900)
    fixed = np.stack([wl.zipf_lists(cfg, s % L, 1, first_token=900 + s // L)[0] for s in range(n_steps)])
    g = np.random.default_rng(31)
    lens = [int(v) for v in g.integers(1, (2 * k if form == 1 else 1800), size=n_steps)]
    lens[5] = 0
    ragged = [np.sort(g.permutation(n)[:c]).astype(np.int32) for c in lens]
    off = np.zeros(n_steps + 1, dtype=np.int32)
    off[1:] = np.cumsum(lens)
    per_layer = np.stack([wl.zipf_lists(cfg, l, 1)[0] for l in range(L)])
    hd = to_dev(heads, cfg.dtype)
    R, N = api.SI_FLAG_RESIDUAL, api.SI_FLAG_PRENORM
    cases = [
        ("fixed", torch.from_numpy(fixed).cuda(), None, k, 0, [fixed[s] for s in range(n_steps)]),
        ("fixed, pre-norm + residual", torch.from_numpy(fixed).cuda(), None, k, R | N, [fixed[s] for s in range(n_steps)]),
        ("offsets, residual", torch.from_numpy(np.concatenate(ragged + [np.zeros(4, np.int32)])).cuda(),
         torch.from_numpy(off).cuda(), max(lens), R, ragged),
        ("per layer, pre-norm", torch.from_numpy(per_layer).cuda(), None, k, N | api.SI_FLAG_LIST_PER_LAYER,
         [per_layer[s % L] for s in range(n_steps)]),
    ]
    for name, idx, offsets, kk, flags, lists in cases:
        y, xn, st = _run_chain(api, m, n_steps, L, hd, idx, offsets, kk, flags, want_xn=True, chain_form=form)
        assert st == 0, (name, api.strerror(st))
        _check_steps_fed_with_device_inputs(api, m, y, xn if flags & N else None, heads, lists, L, flags,
                                            range(n_steps), lambda s: s % L)
        # shallower rings change the timing of everything, not the result
        y2, _, st = _run_chain(api, m, n_steps, L, hd, idx, offsets, kk, flags, ring_stages=2, chain_form=form)
        assert st == 0 and torch.equal(y, y2), name


def test_c2_full_size_chained_sampled(api):
    """Config 2 as the benchmark chains it: 128 tokens, each a chain through all 32 layers with pre-norm and
    residual, 4096 steps in one launch.  Sampled steps are checked against the oracle fed with the input the
    device read; every output must be finite and the hidden state must stay in a sane range."""
    cfg = wl.CONFIGS["c2"]
    keep = (0, 1, 16, 31)
    m = LoadedModel(cfg, keep_layers=keep)
    L, tokens, k = cfg.n_layers, cfg.tokens, cfg.k_active
    n_steps = L * tokens
    heads = wl.x_tokens(cfg, 0, tokens)
    lists = np.empty((tokens, L, k), dtype=np.int32)
    for l in range(L):
        lists[:, l] = wl.zipf_lists(cfg, l, tokens)
    lists = lists.reshape(n_steps, k)
    flags = api.SI_FLAG_RESIDUAL | api.SI_FLAG_PRENORM
    y, xn, st = _run_chain(api, m, n_steps, L, to_dev(heads, cfg.dtype), torch.from_numpy(lists).cuda(), None, k, flags,
                           want_xn=True)
    assert st == 0, api.strerror(st)
    yf = y.float()
    assert bool(torch.isfinite(yf).all())
    rms = yf.pow(2).mean(dim=1).sqrt()
    assert float(rms.max()) < 50.0 and float(rms.min()) > 0.5           # sqrt(1 + 0.6 l)-like growth, no blow-up, no collapse
    steps = [t * L + l for t in (0, 77, 127) for l in keep]
    _check_steps_fed_with_device_inputs(api, m, y, xn, heads, lists, L, flags, steps, lambda s: s % L)
    y2, _, st = _run_chain(api, m, n_steps, L, to_dev(heads, cfg.dtype), torch.from_numpy(lists).cuda(), None, k, flags)
    assert st == 0 and torch.equal(y, y2)


def test_chained_launch_without_weight_copies_ends_cleanly_and_the_next_call_is_correct(api):
    """The diagnostics launch that copies neither records nor down slices (skip_mask bits 3 and 4: the
    bench times it for the cost of the exchanges alone): it must end with status 0 whatever garbage it
    computes, and an ordinary launch on the same workspace right after it must be correct."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=2)
    L, tokens, k = 2, 4, cfg.k_active
    n_steps = L * tokens
    heads = wl.x_tokens(cfg, 0, tokens, first_token=300)
    lists = np.stack([wl.zipf_lists(cfg, s % L, 1, first_token=300 + s // L)[0] for s in range(n_steps)])
    hd, idx = to_dev(heads, cfg.dtype), torch.from_numpy(lists).cuda()
    flags = api.SI_FLAG_RESIDUAL | api.SI_FLAG_PRENORM
    for mask in (8, 16, 24):
        _, _, st = _run_chain(api, m, n_steps, L, hd, idx, None, k, flags, skip_mask=mask, chain_form=2)
        assert st == 0, (mask, api.strerror(st))
    y, xn, st = _run_chain(api, m, n_steps, L, hd, idx, None, k, flags, want_xn=True)
    assert st == 0, api.strerror(st)
    _check_steps_fed_with_device_inputs(api, m, y, xn, heads, [lists[s] for s in range(n_steps)], L, flags,
                                        range(n_steps), lambda s: s % L)


def test_chain_argument_errors(api):
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    k = cfg.k_active
    heads = to_dev(wl.x_tokens(cfg, 0, 2), cfg.dtype)
    idx = torch.from_numpy(wl.zipf_lists(cfg, 0, 4, slot_of_rank=m.slot_of_rank[0])).cuda()
    ws = m.store.workspace(1, k, 4)
    y16 = torch.empty(4, cfg.d_model, dtype=torch.float16, device="cuda")

    def status_of(fn):
        with pytest.raises(api.SelectInferError) as e:
            fn()
        return e.value.status

    h = m.store.handle
    assert status_of(lambda: api.si_decode_chain_forward(h, 4, [0] * 4, 0, heads, idx, None, k, y16, None, EPS, 0, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_decode_chain_forward(h, 4, [0] * 4, 2, heads, idx, None, k, y16, None, EPS,
                                                         api.SI_FLAG_STEPS_ANY_ORDER, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_decode_chain_forward(h, 4, [0, 0, 1, 0], 2, heads, idx, None, k, y16, None, EPS, 0, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_decode_chain_forward(h, 4, [0] * 4, 2, heads, idx, None, k, y16, None, -1.0,
                                                         api.SI_FLAG_PRENORM, ws)) == api.SI_ERR_INVALID_ARG
    assert status_of(lambda: api.si_decode_chain_forward(h, 4, [0] * 4, 2, heads, idx, None, k, y16, None, EPS, 0, ws[:512])) == api.SI_ERR_NOMEM


# ------------------------------------------------------------------ bounded waits that run out

@pytest.mark.parametrize("chained", [False, True])
def test_decode_wait_runs_out_and_the_next_call_is_correct(api, chained):
    """The producer warp of one SM withholds a record, so that SM's consumers wait for something that never
    comes.  With a limit of two million cycles (about a millisecond) the wait runs out: the status word
    reads SI_ERR_TIMEOUT, the launch returns, and an ordinary call on the same workspace right after it is
    correct.  Nothing faults and no wait is unbounded."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    n_steps, k = 12, cfg.k_active
    lists = wl.zipf_lists(cfg, 0, n_steps, slot_of_rank=m.slot_of_rank[0])
    x = wl.x_tokens(cfg, 0, n_steps)
    xd, idx = to_dev(x, cfg.dtype), torch.from_numpy(lists).cuda()
    ws = m.store.workspace(1, k, n_steps)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.zeros(n_steps, cfg.d_model, dtype=torch.float16, device="cuda")
    if chained:
        api.si_debug_decode_chain_forward(m.store.handle, n_steps, [0] * n_steps, 4, xd[:3], idx, None, k, y, None, EPS, 0,
                                          ws, st, withhold=1, wait_cycles=2_000_000)
    else:
        api.si_debug_decode_stack_forward(m.store.handle, n_steps, [0] * n_steps, xd, idx, None, k, y, 0, ws, st,
                                          withhold=1, wait_cycles=2_000_000)
    torch.cuda.synchronize()                                  # returns: the launch ended by itself
    assert st.item() == api.SI_ERR_TIMEOUT
    # the same workspace, an ordinary call: correct
    st.zero_()
    y32 = torch.empty(n_steps, cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_decode_stack_forward(m.store.handle, n_steps, [0] * n_steps, xd, idx, None, k, y32, 0, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for t in (0, 5, n_steps - 1):
        assert_close(from_dev(y32[t]), m.oracle_y(0, x[t], lists[t]), f"after the time-out, step {t}")


@pytest.mark.parametrize("T,prefix", [(8, False), (200, False), (200, True)])
def test_contraction_wait_runs_out_and_the_next_call_is_correct(api, T, prefix):
    """The same for the tensor-core path: one operand tile of the first gate/up CTA is never loaded, its
    MMA-issuing thread gives up after a few thousand probes, the kernels record SI_ERR_TIMEOUT, give their
    tensor memory back and return; the next call on the same workspace is correct.  8 tokens: the one-CTA
    kernels; 200 tokens: the CTA-pair kernels, with gathered weight rows (own lists) and with weight tiles
    fetched by tensor copies (a shared prefix list) -- there the CTA that issues the pair's MMAs gives up,
    tells both CTAs so, and the pair leaves together."""
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg)
    k = cfg.k_active
    if prefix:
        lists = np.tile(np.arange(k, dtype=np.int32), (T, 1))
        flat, flags = lists[0].copy(), api.SI_FLAG_SHARED_LIST
    else:
        lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=m.slot_of_rank[0])
        flat, flags = lists, api.SI_FLAG_UNION_PATH
    x = wl.x_tokens(cfg, 0, T)
    xd, idx = to_dev(x, cfg.dtype), torch.from_numpy(np.ascontiguousarray(flat)).cuda()
    ws = m.store.workspace(T, k, 1)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(T, cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_debug_ffn_forward_waits(m.store.handle, 0, xd, T, idx, None, k, y, flags, ws, st,
                                   spin_limit=20_000, withhold=1)
    torch.cuda.synchronize()
    assert st.item() == api.SI_ERR_TIMEOUT
    st.zero_()
    api.si_ffn_forward(m.store.handle, 0, xd, T, idx, None, k, y, flags, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for t in sorted({0, 1, T // 2, T - 1}):
        assert_close(from_dev(y[t]), m.oracle_y(0, x[t], lists[t]), f"after the time-out, token {t}")


def test_wide_pair_tiles_wait_runs_out_and_the_next_call_is_correct(api):
    """300 tokens over all loaded neurons of a 7B-shaped layer: gate/up tiles of two sub-tiles (two accumulators per
    CTA) and a down contraction whose K is split between two pairs of a cluster of four.  The first pair's first X
    tile is withheld: SI_ERR_TIMEOUT, a clean return, and a correct call afterwards."""
    cfg = wl.CONFIGS["c2"]
    m = LoadedModel(cfg, n_layers=1)
    T, k = 300, cfg.n_loaded
    shared = np.arange(k, dtype=np.int32)
    x = wl.x_tokens(cfg, 0, T)
    xd, idx = to_dev(x, cfg.dtype), torch.from_numpy(shared).cuda()
    ws = m.store.workspace(T, k, 1)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.empty(T, cfg.d_model, dtype=torch.float32, device="cuda")
    api.si_debug_ffn_forward_waits(m.store.handle, 0, xd, T, idx, None, k, y, api.SI_FLAG_SHARED_LIST, ws, st,
                                   spin_limit=20_000, withhold=1)
    torch.cuda.synchronize()
    assert st.item() == api.SI_ERR_TIMEOUT
    st.zero_()
    api.si_ffn_forward(m.store.handle, 0, xd, T, idx, None, k, y, api.SI_FLAG_SHARED_LIST, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for t in (0, 255, 299):
        assert_close(from_dev(y[t]), m.oracle_y(0, x[t], shared), f"after the time-out, token {t}")
