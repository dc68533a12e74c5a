"""GPU parity: offline profiler (Eq. 1 scores, merge, ranking) and the load set, bit-exact against the oracle."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def test_scores_merge_rank_are_bit_exact(api):
    g = np.random.default_rng(21)
    n = 2753                                     # several blocks and a ragged tail
    prompts = [g.standard_normal((T, n)).astype(np.float32) * g.uniform(0.1, 3.0, size=n).astype(np.float32)
               for T in (37, 5, 130)]
    prompts[1][2, 7] = np.float32(0.0)
    files_ref, files_dev = [], []
    for group in ([0, 1], [2]):                  # two score files: prompts 0 + 1, prompt 2
        s_ref, s_dev = None, torch.zeros(n, dtype=torch.float64, device="cuda")
        tokens = 0
        for pi in group:
            s_ref = so.profile_scores(prompts[pi], s_ref)
            api.si_profile_accumulate(torch.from_numpy(prompts[pi]).cuda(), s_dev)
            tokens += prompts[pi].shape[0]
        torch.cuda.synchronize()
        assert np.array_equal(s_dev.cpu().numpy(), s_ref), "Eq. 1 totals differ"
        files_ref.append((s_ref, tokens)); files_dev.append((s_dev, tokens))
    merged_ref = so.merge_scores(files_ref)
    merged = torch.zeros(n, dtype=torch.float64, device="cuda")
    for s_dev, tokens in files_dev:
        api.si_profile_merge(merged, s_dev, tokens)
    rank = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    api.si_profile_rank(merged, rank)
    torch.cuda.synchronize()
    assert np.array_equal(merged.cpu().numpy(), merged_ref)
    assert np.array_equal(rank.cpu().numpy(), so.ranking(merged_ref))


def test_rank_ties_and_nan(api):
    s = np.array([1.0, 3.0, 3.0, np.nan, 0.0, 7.0, 3.0, np.nan, -0.0], dtype=np.float64)
    rank = torch.empty(len(s), dtype=torch.int32, device="cuda")
    api.si_profile_rank(torch.from_numpy(s).cuda(), rank)
    torch.cuda.synchronize()
    assert np.array_equal(rank.cpu().numpy(), so.ranking(s))
    same = np.zeros(3000)
    rank = torch.empty(3000, dtype=torch.int32, device="cuda")
    api.si_profile_rank(torch.from_numpy(same).cuda(), rank)
    torch.cuda.synchronize()
    assert np.array_equal(rank.cpu().numpy(), np.arange(3000))


@pytest.mark.parametrize("n,n_base,n_loaded", [(11008, 3302, 7705), (1376, 0, 688), (500, 500, 500), (4097, 10, 4097)])
def test_loadset_matches_oracle(api, n, n_base, n_loaded):
    g = np.random.default_rng(n)
    task = g.permutation(n).astype(np.int32)
    model = g.permutation(n).astype(np.int32)
    ids = torch.full((n_loaded,), -1, dtype=torch.int32, device="cuda")
    ws = torch.empty((n + 31) // 32, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.si_loadset(torch.from_numpy(task).cuda(), torch.from_numpy(model).cuda(), n_base, ids, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert np.array_equal(ids.cpu().numpy(), so.loadset(task, model, n_base, n_loaded))


def test_loadset_reports_malformed_rankings(api):
    n = 64
    task = torch.arange(n, dtype=torch.int32, device="cuda")
    bad = torch.arange(n, dtype=torch.int32, device="cuda"); bad[5] = 99
    short = torch.zeros(n, dtype=torch.int32, device="cuda")         # one neuron repeated: too few distinct ids
    ws = torch.empty(2, dtype=torch.int32, device="cuda")
    for model, code in ((bad, api.SI_ERR_OUT_OF_RANGE), (short, api.SI_ERR_INVALID_ARG)):
        ids = torch.empty(40, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        api.si_loadset(task, model, 10, ids, ws, st)
        torch.cuda.synchronize()
        assert st.item() == code


def test_profile_to_loadset_pipeline_on_a_small_model(api):
    """The offline chain on a small dense layer: activations of ALL neurons for some profiling tokens
    (si_prefill_forward on a store that holds every neuron) -> Eq. 1 scores -> ranking -> load set.
    Every stage is compared with the oracle working from its own float64 activations; the ranking can
    only differ where two scores are closer than the rounding of h to the store dtype."""
    from paper_2607_18081_b200 import workloads as wl
    from tests.gpu_utils import to_dev
    cfg = wl.Config("tinyprof", 91, 256, 400, 1, "bf16", 100, 25, 4, loaded_rule="perm")
    wg, wu, wd = wl.layer_weights(cfg, 0)
    F, d, T = cfg.d_ff, cfg.d_model, 48
    ids_all = np.arange(F, dtype=np.int32)
    store = api.NeuronStore(1, d, F, [F], cfg.dtype)
    store.load(0, to_dev(wg, cfg.dtype), to_dev(wu, cfg.dtype), to_dev(wd, cfg.dtype), ids_all, 0)
    x = wl.x_tokens(cfg, 0, T)
    y = torch.empty(T, d, dtype=torch.bfloat16, device="cuda")
    acts = torch.empty(T, F, dtype=torch.float32, device="cuda")
    idx = torch.empty(F, dtype=torch.int32, device="cuda"); cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    ws = store.workspace(T, F, 1)
    vws = torch.empty(api.si_prefill_vote_workspace_bytes(T, F, 1) + 256, dtype=torch.uint8, device="cuda")
    vws = vws[(-vws.data_ptr()) % 256:]
    api.si_prefill_forward(store.handle, 0, to_dev(x, cfg.dtype), T, y, 1, 0, 0, 0, api.SI_FLAG_SCORE_ABS, idx, cnt, acts, ws, vws)
    scores = torch.zeros(F, dtype=torch.float64, device="cuda")
    api.si_profile_accumulate(acts, scores)
    rank = torch.empty(F, dtype=torch.int32, device="cuda")
    api.si_profile_rank(scores, rank)
    n_base, n_loaded = F // 5, F // 2
    out = torch.empty(n_loaded, dtype=torch.int32, device="cuda")
    lws = torch.empty((F + 31) // 32, dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.si_loadset(rank, rank, n_base, out, lws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    # oracle chain from its own activations
    h = np.stack([so.ffn(wg, wu, wd, x[t], ids_all, dtype=cfg.dtype, return_h=True)[1] for t in range(T)])
    s_ref = so.profile_scores(h.astype(np.float32))
    assert np.allclose(scores.cpu().numpy(), s_ref, rtol=5e-3)
    r_ref = so.ranking(s_ref)
    ids_ref = so.loadset(r_ref, r_ref, n_base, n_loaded)
    got = out.cpu().numpy()
    assert len(set(got.tolist())) == n_loaded
    assert len(set(got.tolist()) & set(ids_ref.tolist())) >= 0.98 * n_loaded
    # the GPU chain is self-consistent: the load set is the top of its own ranking
    assert np.array_equal(got, rank.cpu().numpy()[:n_loaded])
