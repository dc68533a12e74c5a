"""Pins for the CPU oracle: it is checked against things other than itself before
anything is compared with it -- library float64 routines, closed forms with printed
constants, algebraic invariants, brute force on tiny inputs, and values the paper prints."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.helpers import paper_values


def _rand_problem(seed, d_ff=24, d_model=16, scale=0.5):
    g = np.random.default_rng(seed)
    Wg = g.normal(0, scale, (d_ff, d_model))
    Wu = g.normal(0, scale, (d_ff, d_model))
    Wd = g.normal(0, scale, (d_model, d_ff))
    x = g.normal(0, 1, d_model)
    return Wg, Wu, Wd, x


# ------------------------------------------------------------------ O-FFN

def test_all_neurons_equals_library_dense_swiglu():
    """A = every neuron must be the textbook SwiGLU FFN, evaluated by a float64 library."""
    Wg, Wu, Wd, x = _rand_problem(1, d_ff=96, d_model=64)
    y = so.ffn(Wg, Wu, Wd, x, np.arange(96))
    tWg, tWu, tWd, tx = (torch.from_numpy(a) for a in (Wg, Wu, Wd, x))
    F = torch.nn.functional
    ref = F.linear(F.silu(F.linear(tx, tWg)) * F.linear(tx, tWu), tWd).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)


def test_subset_equals_library_masked_dense():
    """Selective FFN == dense FFN with the unselected activations zeroed (library route)."""
    Wg, Wu, Wd, x = _rand_problem(2, d_ff=96, d_model=64)
    A = np.array([3, 95, 17, 0, 44, 45, 46, 80])
    y = so.ffn(Wg, Wu, Wd, x, A)
    tWg, tWu, tWd, tx = (torch.from_numpy(a) for a in (Wg, Wu, Wd, x))
    F = torch.nn.functional
    h = F.silu(F.linear(tx, tWg)) * F.linear(tx, tWu)
    keep = torch.zeros(96, dtype=torch.float64)
    keep[torch.from_numpy(A)] = 1
    ref = F.linear(h * keep, tWd).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-13)
    # a transposed W_down or swapped gate/up must fail: check they really differ
    wrong = F.linear(F.silu(F.linear(tx, tWu)) * F.linear(tx, tWg) * keep, tWd).numpy()
    assert np.max(np.abs(wrong - ref)) > 1e-3


@pytest.mark.parametrize("seed", [3, 4, 5])
def test_mask_dense_identity_is_exact(seed):
    """Brute force over all neurons with unselected h forced to 0: bit-for-bit equal."""
    Wg, Wu, Wd, x = _rand_problem(seed, d_ff=40, d_model=24)
    g = np.random.default_rng(seed + 100)
    A = g.permutation(40)[: 13]
    keep = np.zeros(40, dtype=np.uint8)
    keep[A] = 1
    y = so.ffn(Wg, Wu, Wd, x, A)
    yb = so.ffn_dense_masked(Wg, Wu, Wd, x, keep)
    assert np.array_equal(y, yb)
    # all neurons selected == dense brute force, exactly
    assert np.array_equal(so.ffn(Wg, Wu, Wd, x, np.arange(40)),
                          so.ffn_dense_masked(Wg, Wu, Wd, x, np.ones(40, np.uint8)))


def test_closed_form_one_hot_neurons():
    """Wg[i]=e_a, Wu[i]=e_b, Wd[:,i]=e_c  =>  y_c = SiLU(x_a) * x_b, with printed SiLU values."""
    silu = {1.0: 0.7310585786300049, -1.0: -0.2689414213699951, 2.0: 1.7615941559557646}
    d_ff, d_model = 6, 5
    for xa, expect in silu.items():
        Wg = np.zeros((d_ff, d_model)); Wu = np.zeros((d_ff, d_model)); Wd = np.zeros((d_model, d_ff))
        a, b, c, i = 1, 3, 4, 2
        Wg[i, a] = 1; Wu[i, b] = 1; Wd[c, i] = 1
        x = np.array([9.0, xa, 7.0, 3.0, -5.0])
        y = so.ffn(Wg, Wu, Wd, x, [i])
        want = np.zeros(d_model); want[c] = expect * 3.0
        np.testing.assert_allclose(y, want, rtol=1e-15, atol=0)
        # the neuron not being selected gives exactly zero
        assert np.array_equal(so.ffn(Wg, Wu, Wd, x, [0, 1, 3]), np.zeros(d_model))
    # independent evaluation of SiLU via math.exp for an odd value
    Wg = np.zeros((2, 2)); Wu = np.zeros((2, 2)); Wd = np.zeros((2, 2))
    Wg[1, 0] = 0.5; Wu[1, 1] = -2.0; Wd[0, 1] = 4.0
    x = np.array([3.0, 0.25])
    g, u = 1.5, -0.5
    want0 = g / (1 + math.exp(-g)) * u * 4.0
    y = so.ffn(Wg, Wu, Wd, x, [1])
    assert y[0] == pytest.approx(want0, rel=1e-15) and y[1] == 0.0


def test_zero_input_and_empty_list():
    Wg, Wu, Wd, x = _rand_problem(6)
    assert np.array_equal(so.ffn(Wg, Wu, Wd, np.zeros_like(x), np.arange(24)), np.zeros(16))
    assert np.array_equal(so.ffn(Wg, Wu, Wd, x, []), np.zeros(16))


def test_additivity_and_order_invariance():
    Wg, Wu, Wd, x = _rand_problem(7, d_ff=60, d_model=32)
    g = np.random.default_rng(70)
    p = g.permutation(60)
    A, B = p[:20], p[20:45]
    yA, yB = so.ffn(Wg, Wu, Wd, x, A), so.ffn(Wg, Wu, Wd, x, B)
    yAB = so.ffn(Wg, Wu, Wd, x, np.concatenate([A, B]))
    np.testing.assert_allclose(yA + yB, yAB, rtol=1e-12, atol=1e-14)
    assert np.array_equal(so.ffn(Wg, Wu, Wd, x, A), so.ffn(Wg, Wu, Wd, x, A[::-1].copy()))
    assert np.array_equal(so.ffn(Wg, Wu, Wd, x, A), so.ffn(Wg, Wu, Wd, x, np.sort(A)))


def test_activation_matches_library_per_neuron():
    """h_i returned by the oracle is SiLU(g_i) * u_i of a float64 library evaluation."""
    Wg, Wu, Wd, x = _rand_problem(8, d_ff=50, d_model=20)
    A = np.array([49, 1, 7, 30])
    _, h = so.ffn(Wg, Wu, Wd, x, A, return_h=True)
    gg = torch.from_numpy(Wg) @ torch.from_numpy(x)
    uu = torch.from_numpy(Wu) @ torch.from_numpy(x)
    ref = (torch.nn.functional.silu(gg) * uu).numpy()[np.sort(A)]
    np.testing.assert_allclose(h, ref, rtol=1e-12)


def test_bad_lists_rejected():
    Wg, Wu, Wd, x = _rand_problem(9)
    with pytest.raises(ValueError):
        so.ffn(Wg, Wu, Wd, x, [1, 1])
    with pytest.raises(ValueError):
        so.ffn(Wg, Wu, Wd, x, [24])
    with pytest.raises(ValueError):
        so.ffn(Wg, Wu, Wd, x, [-1])


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_16bit_widening_is_exact(dtype):
    """Bit patterns go through the oracle's own widening; numpy/torch widen them independently."""
    g = np.random.default_rng(10)
    d_ff, d_model = 32, 24
    mk = lambda shape, s: wl.float_to_bits(g.normal(0, s, shape).astype(np.float32), dtype)
    Wg, Wu, Wd, x = mk((d_ff, d_model), 0.3), mk((d_ff, d_model), 0.3), mk((d_model, d_ff), 0.3), mk((d_model,), 1)
    # include subnormal / tiny / large values in the fp16 case
    if dtype == "f16":
        Wg[0, :4] = np.array([0x0001, 0x03FF, 0x8001, 0x7BFF], dtype=np.uint16)
        x[:4] = np.array([0x3C00, 0x3C00, 0x3C00, 0x0400], dtype=np.uint16)
    A = np.arange(0, d_ff, 3)
    y = so.ffn(Wg, Wu, Wd, x, A, dtype=dtype)
    tdt = torch.float16 if dtype == "f16" else torch.bfloat16
    widen = lambda a: torch.from_numpy(a.view(np.int16)).view(tdt).to(torch.float64).numpy()
    y64 = so.ffn(widen(Wg), widen(Wu), widen(Wd), widen(x), A, dtype="f64")
    assert np.array_equal(y, y64)
    np.testing.assert_array_equal(widen(Wg), wl.bits_to_float64(Wg, dtype))


def test_threads_do_not_change_bits():
    Wg, Wu, Wd, x = _rand_problem(11, d_ff=200, d_model=48)
    A = np.arange(0, 200, 2)
    assert np.array_equal(so.ffn(Wg, Wu, Wd, x, A, threads=1), so.ffn(Wg, Wu, Wd, x, A, threads=4))


def test_tokens_are_independent_masked_union():
    Wg, Wu, Wd, _ = _rand_problem(12, d_ff=30, d_model=12)
    X = np.random.default_rng(13).normal(0, 1, (3, 12))
    lists = [[0, 5, 9], [], [29, 5, 1, 2]]
    Y = so.ffn_tokens(Wg, Wu, Wd, X, lists)
    for t in range(3):
        assert np.array_equal(Y[t], so.ffn(Wg, Wu, Wd, X[t], lists[t]))


# ------------------------------------------------------------------ O-SELECT

def _brute_topk(scores, k):
    """All k-subsets on tiny n: the unique subset consistent with (score desc, index asc)."""
    s = [0.0 if (v == 0) else v for v in np.asarray(scores, np.float32).tolist()]
    n = len(s)
    def better(i, j):
        ni, nj = math.isnan(s[i]), math.isnan(s[j])
        if ni or nj:                       # NaN ranks below every number; NaN vs NaN: index
            return (not ni) or (nj and i < j)
        return s[i] > s[j] or (s[i] == s[j] and i < j)
    good = []
    for sub in itertools.combinations(range(n), k):
        inside = set(sub)
        if all(better(i, j) for i in sub for j in range(n) if j not in inside):
            good.append(sub)
    assert len(good) == 1
    return np.array(good[0], dtype=np.int32)


@pytest.mark.parametrize("scores", [
    [0.5, -1.0, 3.0, 3.0, 0.0, -0.0, 2.0],
    [1.0] * 7,
    [float("nan"), 1.0, float("-inf"), float("inf"), float("nan"), 0.0, -0.0],
    [-3.0, -2.0, -2.0, -2.0, -1.0, -2.0, -5.0],
    [0.0, -0.0, 0.0, -0.0, 0.0, -0.0, 1e-45],
])
def test_topk_against_subset_brute_force(scores):
    for k in range(len(scores) + 1):
        got = so.select_topk(scores, k)
        assert np.array_equal(got, _brute_topk(scores, k)), (scores, k)
        assert got.dtype == np.int32


def test_topk_invariants_random_with_ties():
    g = np.random.default_rng(21)
    for n, k in [(50, 0), (50, 50), (257, 31), (1000, 400)]:
        s = np.round(g.normal(0, 1, n), 1).astype(np.float32)   # many exact ties
        sel = so.select_topk(s, k)
        assert len(sel) == k and np.all(np.diff(sel) > 0)
        inside = np.zeros(n, bool); inside[sel] = True
        if 0 < k < n:
            lo, hi = s[inside].min(), s[~inside].max()
            assert lo >= hi
            if lo == hi:
                assert sel[s[sel] == lo].max() < np.nonzero(~inside & (s == lo))[0].min()
        # library cross-check: stable descending sort
        ref = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k])
        assert np.array_equal(sel, ref)


def test_topk_abs_and_threshold():
    s = np.array([-4.0, 1.0, 3.0, -3.0, 0.5], np.float32)
    assert so.select_topk(s, 2, use_abs=True).tolist() == [0, 2]      # |-3| ties |3|: lower index
    assert so.select_topk(s, 3, use_abs=True).tolist() == [0, 2, 3]
    assert so.select_threshold(s, 0.5).tolist() == [1, 2]
    assert so.select_threshold(s, 0.5, use_abs=True).tolist() == [0, 1, 2, 3]
    assert so.select_threshold([float("nan"), 1.0], -10).tolist() == [1]


# ------------------------------------------------------------------ O-UNION / O-LOADSET

def test_union_brute_force():
    g = np.random.default_rng(31)
    lists = [np.sort(g.permutation(100)[:30]).astype(np.int32) for _ in range(5)]
    U, mask, overlap, cover = so.union(lists, 100)
    assert U.tolist() == sorted(set(np.concatenate(lists).tolist()))
    assert sum(bin(int(w)).count("1") for w in mask.ravel()) == 150
    for t, l in enumerate(lists):
        members = [int(U[p]) for p in range(len(U)) if (int(mask[t, p >> 5]) >> (p & 31)) & 1]
        assert members == l.tolist()
    assert overlap == pytest.approx(1 - len(U) / 150) and cover == pytest.approx(len(U) / 100)


def test_loadset_tiny_and_table1_arithmetic():
    pv = paper_values()
    # Table 1: base 30 % + secondary 40 % = loaded 70 %; static 30 % + dynamic 10 % = computed 40 %
    assert pv["table1_base_pct"] + pv["table1_secondary_pct"] == pv["table1_loaded_pct"]
    assert pv["table1_base_pct"] + pv["table1_dynamic_pct"] == pv["table1_computed_pct"]
    task = [4, 2, 9, 0, 1, 3, 5, 6, 7, 8]
    model = [2, 7, 4, 5, 0, 9, 1, 3, 6, 8]
    got = so.loadset(task, model, n_base=3, n_loaded=7)
    assert got.tolist() == [4, 2, 9, 7, 5, 0, 1]       # 2, 4, 9 skipped in the model ranking
    F = 11008
    nb, nl = so.count_from_pct(30, F), so.count_from_pct(70, F)
    g = np.random.default_rng(41)
    ids = so.loadset(g.permutation(F), g.permutation(F), nb, nl)
    assert len(ids) == nl == 7705 and len(set(ids.tolist())) == nl and nb == 3302


def test_eq2_worked_example_and_layer_range():
    pv = paper_values()
    saving = so.memory_saving(pv["eq2_n_ffn"], pv["eq2_r_load"], pv["eq2_r_layer"], pv["eq2_bytes_per_param"])
    assert saving / 1e9 == pytest.approx(pv["eq2_saving_gb"], rel=1e-12)
    orig, sel = pv["table5_llama32_3b_original_gb"], pv["table5_llama32_3b_selectinfer_gb"]
    assert round(100 * (orig - sel) / orig, 1) == pv["table5_saving_pct"]
    assert abs((orig - sel) - pv["eq2_saving_gb"]) < 0.05          # "aligning with the value observed"
    first, last = int(pv["table1_first_layer"]), int(pv["table1_last_layer"])
    assert len(so.layer_range(int(pv["llama32_1b_layers"]), first, last)) == pv["llama32_1b_selective_layers"]
    n3b = int(pv["llama32_3b_layers"])
    assert len(so.layer_range(n3b, first, last)) / n3b == pv["eq2_r_layer"]
    # Llama3.2-3B FFN parameter count ~ 2.1 B (3 matrices, d_model 3072, d_ff 8192, 28 layers)
    assert round(3 * 3072 * 8192 * 28 / 1e9, 1) == pv["eq2_n_ffn"] / 1e9


def test_count_rounding_of_configs():
    assert wl.CONFIGS["c1"].n_loaded == 688 and wl.CONFIGS["c1"].k_active == 172
    assert wl.CONFIGS["c2"].n_loaded == 7705 and wl.CONFIGS["c2"].k_active == 1541
    assert wl.CONFIGS["c4"].k_active == 3082
    got = [[so.count_from_pct(a, so.count_from_pct(l, 14336)) for a in wl.C5_ACTIVE] for l in wl.C5_LOADED]
    assert got == [[215, 430, 860, 2150], [358, 716, 1433, 3584], [501, 1003, 2007, 5017], [716, 1433, 2867, 7168]]


# --------------------------------------------------------------------------- prefill vote (Section 5)

def test_prefill_vote_worked_example():
    """Hand-worked case.  4 tokens, 6 loaded neurons, alpha = 2: the per-token top-2 lists by |a| are
    {1,4}, {4,5}, {1,4}, {0,5}, hence the counts [1, 2, 0, 0, 3, 2]."""
    acts = np.array([[0.1, -9.0, 0.2, 0.0, 8.0, 0.3],      # |a|: top 2 = {1, 4}
                     [0.1, 0.2, 0.3, 0.0, -7.0, 6.0],      # {4, 5}
                     [0.0, 5.0, 0.1, 0.2, 5.5, 0.3],       # {1, 4}
                     [-4.0, 0.1, 0.2, 0.3, 0.0, 3.0]],     # {0, 5}
                    dtype=np.float32)
    chosen, counts = so.prefill_vote(acts, alpha=2, beta=3, n_static=1, phi_count=3)
    assert counts.tolist() == [1, 2, 0, 0, 3, 2]
    # frequency order: 4 (3), 1 (2), 5 (2), 0 (1) ... ; beta = 3 candidates {4, 1, 5}; static = {0};
    # phi = 3 -> static 0 plus the two most frequent candidates 4 and 1
    assert chosen.tolist() == [0, 1, 4]
    # with n_static = 2 slot 1 is static already: the walk skips it and takes 4, then 5
    chosen, _ = so.prefill_vote(acts, alpha=2, beta=3, n_static=2, phi_count=4)
    assert chosen.tolist() == [0, 1, 4, 5]
    # signed ranking: token 0's top 2 become {4, 5}, token 1's {2, 5}, token 3's {3, 5}
    chosen, counts = so.prefill_vote(acts, alpha=2, beta=2, n_static=0, phi_count=2, use_abs=False)
    assert counts.tolist() == [0, 1, 1, 1, 2, 3] and chosen.tolist() == [4, 5]


def test_prefill_vote_special_cases_and_invariants():
    g = np.random.default_rng(77)
    T, n = 9, 40
    acts = g.standard_normal((T, n)).astype(np.float32)
    # beta = 0: nothing dynamic; phi below the static count truncates the static prefix
    assert so.prefill_vote(acts, 5, 0, 7, 20)[0].tolist() == list(range(7))
    assert so.prefill_vote(acts, 5, 10, 7, 4)[0].tolist() == list(range(4))
    # alpha = n: every neuron is in every list, all counts equal T, candidates are the lowest slots
    chosen, counts = so.prefill_vote(acts, n, 12, 3, 10)
    assert set(counts.tolist()) == {T} and chosen.tolist() == list(range(10))
    # one token: the dynamic part is that token's top alpha by |a|, lowest frequency-tied slots first
    one = acts[:1]
    chosen, counts = so.prefill_vote(one, 6, n, 0, 6)
    assert chosen.tolist() == so.select_topk(one[0], 6, use_abs=True).tolist()
    # invariants on random cases: size, static prefix, counts sum, dominance of the chosen candidates
    for trial in range(20):
        alpha, beta = int(g.integers(0, n + 1)), int(g.integers(0, n + 1))
        n_static, phi = int(g.integers(0, n + 1)), int(g.integers(0, n + 1))
        chosen, counts = so.prefill_vote(acts, alpha, beta, n_static, phi)
        assert counts.sum() == T * alpha and len(set(chosen.tolist())) == len(chosen) <= phi
        assert chosen.tolist() == sorted(chosen.tolist())
        assert all(s in chosen for s in range(min(n_static, phi)))
        dyn = [i for i in chosen if i >= n_static]
        assert all(counts[i] > 0 for i in dyn)
        if dyn and len(chosen) == phi:      # a chosen candidate is never less frequent than a left-out neuron
            worst = min((counts[i], -i) for i in dyn)
            top_beta = sorted(range(n), key=lambda i: (-int(counts[i]), i))[:beta]
            left_out = [i for i in top_beta if i >= n_static and i not in dyn and counts[i] > 0]
            assert all((counts[i], -i) < worst for i in left_out)


# --------------------------------------------------------------------------- profiler (Section 3, Eq. 1)

def test_profiler_scores_merge_and_ranking():
    """Eq. 1 on a hand-worked case, additivity over prompts, the merge rule and the ranking's tie-break."""
    a = np.array([[1.0, -2.0, 0.5, 0.0], [-3.0, 2.0, 0.5, -0.0], [0.25, 0.0, -0.5, 0.0]], dtype=np.float32)
    s = so.profile_scores(a)
    assert s.tolist() == [4.25, 4.0, 1.5, 0.0]                       # column sums of |a|
    # scoring a prompt in two pieces gives the same totals as scoring it at once (same order of additions)
    assert np.array_equal(so.profile_scores(a[2:], so.profile_scores(a[:2])), s)
    # Eq. 1 against a library evaluation on random data
    g = np.random.default_rng(3)
    b = g.standard_normal((57, 33)).astype(np.float32)
    assert np.allclose(so.profile_scores(b), np.abs(b.astype(np.float64)).sum(axis=0), rtol=1e-14, atol=0)
    # merge: normalise by token count, then sum -- a file with twice the tokens and twice the scores counts the same
    f1, f2 = (np.array([4.0, 2.0, 0.0]), 2), (np.array([8.0, 4.0, 0.0]), 4)
    assert so.merge_scores([f1]).tolist() == [2.0, 1.0, 0.0]
    assert so.merge_scores([f1, f2]).tolist() == [4.0, 2.0, 0.0]
    with pytest.raises(ValueError):
        so.merge_scores([(np.ones(3), 0)])
    # ranking: decreasing score, ties to the lower index, NaN last
    assert so.ranking(np.array([1.0, 3.0, 3.0, np.nan, 0.0, 7.0])).tolist() == [5, 1, 2, 0, 4, 3]
    r = so.ranking(so.merge_scores([(so.profile_scores(b), 57)]))
    m = so.profile_scores(b)
    assert sorted(r.tolist()) == list(range(33)) and all(m[r[i]] >= m[r[i + 1]] for i in range(32))
    # ranking feeds the load set of Section 4: base neurons from the task ranking come first
    task, model = so.ranking(so.profile_scores(b[:20])), r
    ids = so.loadset(task, model, 5, 12)
    assert ids[:5].tolist() == task[:5].tolist() and len(set(ids.tolist())) == 12


# ---------------------------------------------------------------------------------------------
# Neuron-sharded evaluation: Section 5 writes the layer output as a sum over the selected neurons, so
# partial outputs over disjoint neuron subsets must add up to it.
@pytest.mark.parametrize("world", [1, 2, 3, 5])
def test_shard_partition_and_partial_sums(world):
    Wg, Wu, Wd, x = _rand_problem(21 + world, d_ff=90, d_model=24)
    g = np.random.default_rng(world)
    loaded = g.permutation(90)[:61].astype(np.int32)              # slot -> global neuron id
    lists = [np.sort(g.permutation(61)[:k]).astype(np.int32) for k in (0, 1, 17, 61)]
    # every slot is owned exactly once, local order = global order
    owned = [so.shard_slots(61, r, world) for r in range(world)]
    assert sorted(np.concatenate(owned).tolist()) == list(range(61))
    for r in range(world):
        assert np.all(np.diff(owned[r]) > 0)
    for l in lists:
        parts = [so.shard_lists([l], r, world)[0] for r in range(world)]
        # mapping back local -> global recovers the list, split without loss or duplication
        back = np.sort(np.concatenate([owned[r][parts[r]] for r in range(world)]))
        assert np.array_equal(back, l)
        for r in range(world):
            assert np.all(np.diff(parts[r]) > 0)                   # order kept
        y_full = so.ffn(Wg, Wu, Wd, x, loaded[l])
        y_sum = np.zeros_like(y_full)
        for r in range(world):
            ids_r = loaded[owned[r]]                               # the ids device r loads, in local slot order
            y_sum += so.ffn(Wg, Wu, Wd, x, ids_r[parts[r]])
        np.testing.assert_allclose(y_sum, y_full, rtol=1e-12, atol=1e-14)


def test_shard_lists_hand_example():
    # slots 0..9 on 3 devices: device 0 owns 0,3,6,9; device 1 owns 1,4,7; device 2 owns 2,5,8
    l = np.array([1, 3, 4, 8, 9], dtype=np.int32)
    assert so.shard_lists([l], 0, 3)[0].tolist() == [1, 3]         # slots 3, 9 -> local 1, 3
    assert so.shard_lists([l], 1, 3)[0].tolist() == [0, 1]         # slots 1, 4 -> local 0, 1
    assert so.shard_lists([l], 2, 3)[0].tolist() == [2]            # slot 8 -> local 2
    assert so.shard_slots(10, 1, 3).tolist() == [1, 4, 7]


# ------------------------------------------------------------------ the error measure of the parity tests

def test_error_metrics_hand_worked_values():
    """error_metrics carries every FFN parity assertion, so it is pinned on vectors worked by hand:
    y_ref = (4, -2, 0, 1), y = (4.5, -2, -0.25, 1)  =>  |err| = (0.5, 0, 0.25, 0);
    max|err| / max|y_ref| = 0.5 / 4 = 0.125;  mean|err| / mean|y_ref| = 0.1875 / 1.75 = 3/28.
    The two ratios differ, each differs from the figure a swapped max/mean would give (0.5 / 1.75,
    0.1875 / 4), and normalising by y instead of y_ref would give 0.5 / 4.5."""
    y_ref = np.array([4.0, -2.0, 0.0, 1.0])
    y = np.array([4.5, -2.0, -0.25, 1.0])
    e_max, e_mean = so.error_metrics(y, y_ref)
    assert e_max == 0.125
    assert e_mean == pytest.approx(3.0 / 28.0, rel=1e-15)
    # a negative error counts by its size; the sign of the reference does not matter
    assert so.error_metrics(-y, -y_ref) == (e_max, e_mean)
    assert so.error_metrics(2 * y_ref - y, y_ref) == (e_max, e_mean)
    # the reference normalises, not the value under test
    e2 = so.error_metrics(y_ref, y)
    assert e2[0] == pytest.approx(0.5 / 4.5, rel=1e-15) and e2[1] == pytest.approx(0.1875 / 1.9375, rel=1e-15)
    # exact agreement is exactly zero; one wrong element of many moves the max ratio, barely the mean ratio
    assert so.error_metrics(y_ref, y_ref) == (0.0, 0.0)
    big_ref = np.ones(1000)
    big = big_ref.copy()
    big[123] = 1.5
    e_max, e_mean = so.error_metrics(big, big_ref)
    assert e_max == 0.5 and e_mean == pytest.approx(0.5 / 1000, rel=1e-12)
    # a reference of zeros: the raw errors come back (nothing to divide by)
    assert so.error_metrics(np.array([0.25, -0.5]), np.zeros(2)) == (0.5, 0.375)
    # 16-bit and fp32 inputs are widened, not truncated
    assert so.error_metrics(np.array([1.5], dtype=np.float32), np.array([1.0], dtype=np.float16)) == (0.5, 0.5)


def test_parity_tolerances_are_the_stated_ones():
    """The GPU parity helper uses the stated bounds -- max|err| <= 2e-2 max|y_ref| and
    mean|err| / mean|y_ref| <= 5e-3 per token -- and fails just outside either."""
    from tests import gpu_utils
    assert gpu_utils.MAX_ERR == 2e-2 and gpu_utils.MEAN_REL == 5e-3
    ref = np.ones(100)
    ok = ref.copy(); ok[0] = 1.0 + 1.9e-2                     # max ratio 1.9e-2, mean ratio 1.9e-4
    gpu_utils.assert_close(ok, ref)
    bad_max = ref.copy(); bad_max[0] = 1.0 + 2.1e-2
    with pytest.raises(AssertionError):
        gpu_utils.assert_close(bad_max, ref)
    bad_mean = ref + 5.1e-3                                    # max ratio 5.1e-3 passes, mean ratio 5.1e-3 does not
    with pytest.raises(AssertionError):
        gpu_utils.assert_close(bad_mean, ref)
    gpu_utils.assert_close(ref + 4.9e-3, ref)
    # the tight bound used for fp32 outputs of the decode kernels
    assert gpu_utils.F32_MAX_ERR <= 1e-4
    with pytest.raises(AssertionError):
        gpu_utils.assert_close_f32(ref + 2e-4, ref)
    gpu_utils.assert_close_f32(ref + 1e-6, ref)


# ------------------------------------------------------------------ chained layers: rounding, normalisation, chain

@pytest.mark.parametrize("dtype,tdt", [("bf16", torch.bfloat16), ("f16", torch.float16)])
def test_round_bits_matches_library_rounding(dtype, tdt):
    """Round-to-nearest-even to the 16-bit types against torch's conversion, ties and specials included."""
    g = np.random.default_rng(11)
    v = np.concatenate([g.normal(0, 1, 4000), g.normal(0, 1e-3, 1000), g.normal(0, 300, 1000),
                        [0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 65504.0, 1e-8]])
    if dtype == "bf16":
        # exact ties: 1 + 2^-8 lies halfway between two bf16 values (-> even: 1.0); 1 + 3 * 2^-8 -> 1 + 2^-6
        v = np.concatenate([v, [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8)]])
    else:
        v = np.concatenate([v, [1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 6e-8, 2.0 ** -24, 2.0 ** -25]])
    bits = so.round_bits(v, dtype)
    ref = torch.from_numpy(v.astype(np.float32)).to(tdt).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    # widening is the exact inverse on representable values
    back = so.widen_bits(bits, dtype)
    assert np.array_equal(so.round_bits(back, dtype), bits)
    assert np.array_equal(back, torch.from_numpy(ref.view(np.int16)).view(tdt).to(torch.float64).numpy())
    if dtype == "bf16":
        assert so.widen_bits(so.round_bits([1.0 + 2.0 ** -8], dtype), dtype)[0] == 1.0
        assert so.widen_bits(so.round_bits([1.0 + 3 * 2.0 ** -8], dtype), dtype)[0] == 1.0 + 2.0 ** -6


def test_rmsnorm_closed_forms_and_library():
    """x = (3, 4): mean square 12.5, so the result is (3, 4) / sqrt(12.5); unit RMS after normalising with
    eps = 0; scale invariance; eps in the right place; torch's rms_norm in float64."""
    y = so.rmsnorm([3.0, 4.0], 0.0)
    np.testing.assert_allclose(y, np.array([3.0, 4.0]) / math.sqrt(12.5), rtol=1e-15)
    np.testing.assert_allclose(so.rmsnorm([3.0, 4.0], 3.5), np.array([3.0, 4.0]) / 4.0, rtol=1e-15)   # 12.5 + 3.5 = 16
    g = np.random.default_rng(5)
    x = g.normal(0, 3, 257)
    y = so.rmsnorm(x, 0.0)
    assert abs(np.sqrt(np.mean(y * y)) - 1.0) < 1e-14
    np.testing.assert_allclose(so.rmsnorm(7.5 * x, 0.0), y, rtol=1e-13)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (257,), eps=1e-5).numpy()
    np.testing.assert_allclose(so.rmsnorm(x, 1e-5), ref, rtol=1e-13)
    # a sum in place of the mean, or eps outside the root, must fail: they differ visibly
    assert np.max(np.abs(x / np.sqrt(np.sum(x * x) + 1e-5) - ref)) > 1e-2
    assert np.max(np.abs(x / (np.sqrt(np.mean(x * x)) + 0.5) - so.rmsnorm(x, 0.5))) > 1e-3


def test_ffn_chain_is_the_ffn_applied_step_after_step():
    """The chain against its definition written out with the pinned pieces, on a tiny two-layer model:
    rounding between steps, the residual taken from the step's own input, the normalised row fed to
    the FFN, lists and layers indexed per step."""
    g = np.random.default_rng(21)
    d_ff, d = 20, 16
    mk = lambda *shape: so.round_bits(g.normal(0, 0.4, shape), "bf16")
    weights = [(mk(d_ff, d), mk(d_ff, d), mk(d, d_ff)) for _ in range(2)]
    ids = [g.permutation(d_ff)[:12].astype(np.int32) for _ in range(2)]
    lists = [np.sort(g.permutation(12)[:k]).astype(np.int32) for k in (5, 7, 0, 12)]
    layers = [0, 1, 1, 0]
    x0 = so.round_bits(g.normal(0, 1, d), "bf16")
    for residual in (False, True):
        for prenorm in (False, True):
            out, xn, raw = so.ffn_chain(weights, layers, ids, lists, x0, "bf16", residual=residual, prenorm=prenorm, eps=1e-5)
            cur = x0
            for s in range(4):
                xin = so.widen_bits(cur, "bf16")
                xs = so.round_bits(so.rmsnorm(xin, 1e-5), "bf16") if prenorm else cur
                assert np.array_equal(xn[s], xs)
                wg, wu, wd = weights[layers[s]]
                y = so.ffn(wg, wu, wd, xs, ids[layers[s]][lists[s]], dtype="bf16")
                if residual:
                    y = y + xin
                assert np.array_equal(raw[s], y)
                cur = so.round_bits(y, "bf16")
                assert np.array_equal(out[s], cur)
            # the empty list of step 2: the FFN adds nothing
            assert np.array_equal(raw[2], so.widen_bits(out[1], "bf16") if residual else np.zeros(d))
    # float64 library evaluation of a two-step chain without rounding effects: weights and x chosen so
    # that every intermediate is exactly representable is not possible in general, so compare loosely
    out, _, raw = so.ffn_chain(weights, [0, 1], ids, [np.arange(12), np.arange(12)], x0, "bf16")
    F = torch.nn.functional
    W = [[torch.from_numpy(so.widen_bits(w, "bf16")) for w in ws] for ws in weights]
    def dense(l, v):
        sel = torch.from_numpy(ids[l].astype(np.int64))
        return F.linear(F.silu(F.linear(v, W[l][0][sel])) * F.linear(v, W[l][1][sel]), W[l][2][:, sel])
    y0 = dense(0, torch.from_numpy(so.widen_bits(x0, "bf16")))
    np.testing.assert_allclose(raw[0], y0.numpy(), rtol=1e-12, atol=1e-14)
    y1 = dense(1, torch.from_numpy(so.widen_bits(so.round_bits(y0.numpy(), "bf16"), "bf16")))
    np.testing.assert_allclose(raw[1], y1.numpy(), rtol=1e-12, atol=1e-14)
