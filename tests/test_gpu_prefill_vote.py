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
