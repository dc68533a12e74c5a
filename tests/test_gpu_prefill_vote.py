"""GPU parity: selection of the dynamic neurons during prefill (Section 5) against the oracle, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _vote(api, acts, alpha, beta, n_static, phi, use_abs=True):
    T, n = acts.shape
    a = torch.from_numpy(acts).cuda()
    idx = torch.full((max(phi, 4),), -7, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    counts = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.si_prefill_vote_workspace_bytes(T, n, alpha) + 256, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    api.si_prefill_vote(a, alpha, beta, n_static, phi, api.SI_FLAG_SCORE_ABS if use_abs else 0, idx, cnt, counts, ws)
    torch.cuda.synchronize()
    m = int(cnt[0].item())
    return idx[:m].cpu().numpy(), counts.cpu().numpy()


def _check(api, acts, alpha, beta, n_static, phi, use_abs=True):
    got, got_counts = _vote(api, acts, alpha, beta, n_static, phi, use_abs)
    ref, ref_counts = so.prefill_vote(acts, alpha, beta, n_static, phi, use_abs=use_abs)
    assert np.array_equal(got_counts, ref_counts.astype(np.int32)), "frequencies differ"
    assert np.array_equal(got, ref), (alpha, beta, n_static, phi, use_abs)


def test_vote_small_random_and_degenerate(api):
    g = np.random.default_rng(5)
    T, n = 11, 300
    acts = g.standard_normal((T, n)).astype(np.float32)
    for alpha, beta, n_static, phi in [(30, 50, 20, 60), (30, 50, 0, 25), (1, 1, 0, 1), (300, 40, 10, 45),
                                       (30, 0, 20, 60), (30, 50, 80, 40), (0, 50, 20, 60), (30, 300, 20, 300),
                                       (5, 200, 3, 120)]:
        _check(api, acts, alpha, beta, n_static, phi)
        _check(api, acts, alpha, beta, n_static, phi, use_abs=False)


def test_vote_ties_everywhere(api):
    """Activations from a tiny value set: ties inside the per-token ranking and among the frequencies."""
    g = np.random.default_rng(6)
    T, n = 16, 257
    acts = g.choice(np.array([-2.0, -1.0, -0.0, 0.0, 1.0, 2.0], dtype=np.float32), size=(T, n))
    for alpha, beta, n_static, phi in [(40, 64, 16, 70), (100, 100, 0, 100), (13, 257, 5, 200)]:
        _check(api, acts, alpha, beta, n_static, phi)


def test_vote_prefill_shape_7b(api):
    """Config-4 shape: 512 prompt tokens over 7705 loaded neurons; static = 30 % of d_ff, phi = 40 % of d_ff
    (Table 1), alpha = 20 % of the loaded neurons, beta = 2 * dynamic count."""
    cfg = wl.CONFIGS["c4"]
    T, n = 512, cfg.n_loaded
    g = np.random.default_rng(7)
    # a stable hot core plus noise, so that frequencies are spread between 0 and T
    hot = (1.0 / np.sqrt(1.0 + np.arange(n))).astype(np.float32)
    acts = (g.standard_normal((T, n)).astype(np.float32) * (0.3 + 3.0 * hot)[None, :])
    n_static = (30 * cfg.d_ff) // 100
    phi = (40 * cfg.d_ff) // 100
    _check(api, acts, (20 * n) // 100, 2 * (phi - n_static), n_static, phi)


def _aligned(nbytes):
    t = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    return t[(-t.data_ptr()) % 256:]


@pytest.mark.parametrize("cfg_name,T", [("c1", 24), ("c2", 40)])
def test_prefill_forward_outputs_activations_and_vote(api, cfg_name, T):
    """si_prefill_forward: y over all loaded neurons and the activations against the float64 oracle; the
    chosen slots against si_prefill_vote on the exported activations (same library, same decision
    precision) and, as a sanity check, against the oracle's vote on its own float64 activations."""
    from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev
    cfg = wl.CONFIGS[cfg_name]
    m = LoadedModel(cfg, n_layers=1)
    n, d = cfg.n_loaded, cfg.d_model
    x = wl.x_tokens(cfg, 0, T)
    n_static, phi, alpha = (30 * n) // 100, (45 * n) // 100, (15 * n) // 100
    beta = 2 * (phi - n_static)
    tdt = torch.float16 if cfg.dtype == "f16" else torch.bfloat16
    y = torch.empty(T, d, dtype=tdt, device="cuda")
    acts = torch.empty(T, n, dtype=torch.float32, device="cuda")
    idx = torch.full((phi,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = m.store.workspace(T, n, 1)
    vws = _aligned(api.si_prefill_vote_workspace_bytes(T, n, alpha))
    api.si_prefill_forward(m.store.handle, 0, to_dev(x, cfg.dtype), T, y, alpha, beta, n_static, phi,
                           api.SI_FLAG_SCORE_ABS, idx, cnt, acts, ws, vws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    wg, wu, wd = m.host[0]
    gids = m.ids[0]                                  # global neuron id of every slot
    slot_of_sorted = np.argsort(gids, kind="stable")  # the oracle reports h for the ids in ascending order
    h_ref = np.empty((T, n))
    for t in range(T):
        y_ref, h = so.ffn(wg, wu, wd, x[t], gids, dtype=cfg.dtype, threads=so.host_threads(), return_h=True)
        h_ref[t, slot_of_sorted] = h
        assert_close(from_dev(y[t]), y_ref, f"{cfg_name} prefill token {t}")
    # activations: fp32-accumulated tensor-core dot products rounded to the store dtype
    a = acts.cpu().numpy().astype(np.float64)
    rel = np.abs(a - h_ref).max() / np.abs(h_ref).max()
    assert rel <= (2e-3 if cfg.dtype == "f16" else 1e-2), rel
    # the decision: identical to the standalone vote on the exported activations
    idx2 = torch.full((phi,), -1, dtype=torch.int32, device="cuda")
    cnt2 = torch.zeros(4, dtype=torch.int32, device="cuda")
    api.si_prefill_vote(acts, alpha, beta, n_static, phi, api.SI_FLAG_SCORE_ABS, idx2, cnt2, None, vws)
    torch.cuda.synchronize()
    k = int(cnt[0].item())
    assert k == int(cnt2[0].item()) and torch.equal(idx[:k], idx2[:k])
    # and close to the oracle's own end-to-end answer (rounding can only flip near-ties)
    ref, _ = so.prefill_vote(h_ref.astype(np.float32), alpha, beta, n_static, phi, use_abs=True)
    got = set(idx[:k].cpu().numpy().tolist())
    inter = len(got & set(ref.tolist()))
    assert k == len(ref) and inter >= 0.97 * len(ref), (k, len(ref), inter)


@pytest.mark.parametrize("T", [1, 3, 129])
def test_prefill_forward_short_and_odd_prompts(api, T):
    """A one-token prompt, an odd handful, and one token past a 128-wide token tile."""
    from tests.gpu_utils import LoadedModel, assert_close, from_dev, to_dev
    cfg = wl.CONFIGS["c1"]
    m = LoadedModel(cfg, n_layers=1)
    n, d = cfg.n_loaded, cfg.d_model
    x = wl.x_tokens(cfg, 0, T)
    y = torch.empty(T, d, dtype=torch.float16, device="cuda")
    idx = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    acts = torch.empty(T, n, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = m.store.workspace(max(T, 2), n, 1)
    vws = _aligned(api.si_prefill_vote_workspace_bytes(T, n, 50))
    api.si_prefill_forward(m.store.handle, 0, to_dev(x, cfg.dtype), T, y, 50, 200, 100, 250, api.SI_FLAG_SCORE_ABS,
                           idx, cnt, acts, ws, vws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    for t in sorted({0, T - 1}):
        assert_close(from_dev(y[t]), m.oracle_y(0, x[t], np.arange(n)), f"T={T} token {t}")
    k = int(cnt[0].item())
    got = idx[:k].cpu().numpy()
    assert 100 <= k <= 250 and np.array_equal(got[:100], np.arange(100)) and np.all(np.diff(got) > 0)
    # with one token every candidate occurs exactly once: the dynamic part is a subset of that token's top alpha
    if T == 1:
        a = np.abs(acts[0].cpu().numpy())
        top = np.argsort(-a, kind="stable")[:50]          # the exported activations, ranked by a library sort
        assert set(got[100:].tolist()) <= set(top.tolist())
