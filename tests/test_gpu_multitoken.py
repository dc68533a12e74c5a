"""GPU parity: union builder (bit-exact) and the multi-token tensor-core path vs the oracle."""
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


@pytest.fixture(scope="module")
def c1(api):
    return LoadedModel(wl.CONFIGS["c1"])


@pytest.fixture(scope="module")
def m7b(api):
    return LoadedModel(wl.CONFIGS["c2"], n_layers=1)


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def _run(api, m, layer, x_bits, lists_flat, offsets, k_fixed, T, flags=0, y_dtype=torch.float32):
    cfg = m.cfg
    ws = m.store.workspace(max(T, 2), max(k_fixed, 1), 1)       # (the union path's regions exist from T_max = 2 on)
    y = torch.full((T, cfg.d_model), 3.0, dtype=y_dtype, device="cuda")
    st = _status()
    idx = torch.from_numpy(np.ascontiguousarray(lists_flat, dtype=np.int32)).cuda()
    off = None if offsets is None else torch.from_numpy(np.ascontiguousarray(offsets, dtype=np.int32)).cuda()
    api.si_ffn_forward(m.store.handle, layer, to_dev(x_bits, cfg.dtype), T, idx, off, k_fixed, y, flags, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0, api.strerror(int(st.item()))
    return y


def test_union_is_bit_exact(api, c1):
    cfg = c1.cfg
    T, k = 5, cfg.k_active
    lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=c1.slot_of_rank[0])
    ws = c1.store.workspace(T, k, 1)
    uni = torch.full((cfg.n_loaded,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    api.si_union(c1.store.handle, 0, T, torch.from_numpy(lists).cuda(), None, k, uni, cnt, ws)
    torch.cuda.synchronize()
    U, mask, overlap, cover = so.union(lists, cfg.n_loaded)
    n = int(cnt[0].item())
    assert n == len(U) and np.array_equal(uni[:n].cpu().numpy(), U)
    assert 0.0 < overlap < 1.0 and cover <= 1.0


@pytest.mark.parametrize("T", [2, 4, 16])
def test_c1_multitoken_matches_per_token_oracle(api, c1, T):
    """A few tokens, with and without the flag that forces the union path (which every call with more than one token
    takes anyway)."""
    cfg = c1.cfg
    lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=c1.slot_of_rank[0])
    x = wl.x_tokens(cfg, 0, T)
    for flags in (0, api.SI_FLAG_UNION_PATH):
        y = _run(api, c1, 0, x, lists, None, cfg.k_active, T, flags=flags)
        for t in range(T):
            assert_close(from_dev(y[t]), c1.oracle_y(0, x[t], lists[t]), f"T={T} token {t} flags={flags}")


def test_c1_ragged_empty_unmasked_residual(api, c1):
    cfg = c1.cfg
    n = cfg.n_loaded
    g = np.random.default_rng(9)
    lens = [40, 0, 200, n, 1]
    T = len(lens)
    lists = [np.sort(g.permutation(n)[:k]).astype(np.int32) for k in lens]
    offsets = np.zeros(T + 1, np.int32); offsets[1:] = np.cumsum(lens)
    x = wl.x_tokens(cfg, 0, T, first_token=50)
    flat = np.concatenate(lists)
    y = _run(api, c1, 0, x, flat, offsets, n, T, flags=api.SI_FLAG_RESIDUAL | api.SI_FLAG_CHECK)
    for t in range(T):
        ref = c1.oracle_y(0, x[t], lists[t]) + wl.bits_to_float64(x[t], cfg.dtype)
        assert_close(from_dev(y[t]), ref, f"ragged token {t}")
    # token 1 has an empty list: exactly x
    assert np.array_equal(from_dev(y[1]), wl.bits_to_float64(x[1], cfg.dtype))
    # unmasked extension: every token uses the whole union
    lists3 = [lists[0], lists[2], lists[4]]
    off3 = np.array([0, 40, 240, 241], np.int32)
    U, _, _, _ = so.union(lists3, n)
    y = _run(api, c1, 0, x[:3], np.concatenate(lists3), off3, n, 3, flags=api.SI_FLAG_UNION_UNMASKED)
    for t in range(3):
        assert_close(from_dev(y[t]), c1.oracle_y(0, x[t], U), f"unmasked token {t}")


def _slots_of_bitmap(row: np.ndarray) -> np.ndarray:
    bits = np.unpackbits(row.view(np.uint8), bitorder="little")
    return np.nonzero(bits)[0].astype(np.int32)


@pytest.mark.parametrize("which,T", [("c1", 5), ("c1", 40), ("7b", 1), ("7b", 8), ("7b", 16), ("7b", 32)])
def test_union_and_token_bitmaps_are_bit_exact(api, c1, m7b, which, T):
    """What the union stage leaves for the contractions -- the ascending union and one slot bitmap per
    token, which decides the union entries a token uses (masked semantics) -- against the oracle's union
    and membership masks, for the one-block kernel (few entries) and the several-block kernel."""
    m = c1 if which == "c1" else m7b
    cfg = m.cfg
    k, n = cfg.k_active, cfg.n_loaded
    lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=m.slot_of_rank[0], first_token=11)
    ws = m.store.workspace(max(T, 2), k, 1)
    mask_words = (n + 127) // 128 * 4
    uni = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(4, dtype=torch.int32, device="cuda")
    masks = torch.full((T, mask_words), -1, dtype=torch.int32, device="cuda")
    api.si_debug_union_masks(m.store.handle, 0, T, torch.from_numpy(lists).cuda(), None, k, uni, cnt, masks, ws)
    torch.cuda.synchronize()
    U, omask, _, _ = so.union(lists, n)
    nu = int(cnt[0].item())
    assert nu == len(U) and np.array_equal(uni[:nu].cpu().numpy(), U)
    got = masks.cpu().numpy().view(np.uint32)
    for t in range(T):
        mine = _slots_of_bitmap(got[t])
        # the oracle's mask is over positions in U: translate to slots
        theirs = U[_slots_of_bitmap(omask[t])]
        assert np.array_equal(mine, theirs), f"token {t}"
        assert np.array_equal(mine, np.sort(lists[t]))
    assert sum(len(_slots_of_bitmap(got[t])) for t in range(T)) == T * k


@pytest.mark.parametrize("T", [1, 4, 8, 16, 32])
def test_7b_batched_decode_union(api, m7b, T):
    """Config-3 shape: T tokens with independent Zipf lists over a 7B-shaped layer, every batch size of the
    configuration (a single token is forced onto the union path)."""
    cfg = m7b.cfg
    k = cfg.k_active
    lists = wl.zipf_lists(cfg, 0, T)
    x = wl.x_tokens(cfg, 0, T)
    y = _run(api, m7b, 0, x, lists, None, k, T, flags=api.SI_FLAG_UNION_PATH)
    yb = _run(api, m7b, 0, x, lists, None, k, T, y_dtype=torch.bfloat16)
    for t in sorted({0, min(1, T - 1), T // 2, T - 1}):
        ref = m7b.oracle_y(0, x[t], lists[t])
        assert_close(from_dev(y[t]), ref, f"T={T} token {t}")
        assert_close(from_dev(yb[t]), ref, f"T={T} token {t} bf16 out")
    # run-to-run bit stability
    y2 = _run(api, m7b, 0, x, lists, None, k, T, flags=api.SI_FLAG_UNION_PATH)
    assert torch.equal(y, y2)


def test_7b_prefill_shared_list(api, m7b):
    """Config-4 shape: 512 tokens, one shared list = the first 40 % of the loaded slots."""
    cfg = wl.CONFIGS["c4"]
    T, k = 512, cfg.k_active
    assert k == 3082
    shared = np.arange(k, dtype=np.int32)
    x = wl.x_tokens(cfg, 0, T)
    y = _run(api, m7b, 0, x, shared, None, k, T, flags=api.SI_FLAG_SHARED_LIST)
    for t in (0, 17, 255, 256, 300, 511):
        # the model was loaded from the c2 recipe; the oracle uses that model's weights
        ref = m7b.oracle_y(0, x[t], shared)
        assert_close(from_dev(y[t]), ref, f"prefill token {t}")


def test_7b_many_tokens_own_lists_residual(api, m7b):
    """300 tokens with lists of their own (more than 128 tokens: the contractions run on CTA pairs, 256 tokens
    per pair): the union covers nearly the whole loaded set, every token keeps to its own list through its
    slot bitmap, the second token tile is ragged."""
    cfg = m7b.cfg
    T, k = 300, cfg.k_active
    lists = wl.zipf_lists(cfg, 0, T)
    x = wl.x_tokens(cfg, 0, T)
    y = _run(api, m7b, 0, x, lists, None, k, T, flags=api.SI_FLAG_RESIDUAL, y_dtype=torch.bfloat16)
    for t in (0, 128, 255, 256, 299):
        ref = m7b.oracle_y(0, x[t], lists[t]) + wl.bits_to_float64(x[t], cfg.dtype)
        assert_close(from_dev(y[t]), ref, f"300-token batch, token {t}")


@pytest.mark.parametrize("T", [130, 200])
def test_c1_many_tokens_narrow_token_tiles(api, c1, T):
    """More than 128 tokens over a small layer (CTA pairs, one ragged tile of 256 tokens): ragged lists with an
    empty one, then a shared list of scattered slots (gathered weight rows), fp16 output."""
    cfg = c1.cfg
    n = cfg.n_loaded
    g = np.random.default_rng(100 + T)
    lens = g.integers(0, n // 2, size=T)
    lens[3] = 0
    lists = [np.sort(g.permutation(n)[:k]).astype(np.int32) for k in lens]
    offsets = np.zeros(T + 1, np.int32); offsets[1:] = np.cumsum(lens)
    x = wl.x_tokens(cfg, 0, T, first_token=7)
    y = _run(api, c1, 0, x, np.concatenate(lists), offsets, n, T)
    for t in (0, 3, 64, 127, 128, T - 1):
        assert_close(from_dev(y[t]), c1.oracle_y(0, x[t], lists[t]), f"T={T} token {t}")
    # one shared list for all tokens
    shared = np.sort(g.permutation(n)[: n // 3]).astype(np.int32)
    y = _run(api, c1, 0, x, shared, None, len(shared), T, flags=api.SI_FLAG_SHARED_LIST, y_dtype=torch.float16)
    for t in (0, 127, 128, T - 1):
        assert_close(from_dev(y[t]), c1.oracle_y(0, x[t], shared), f"shared list, T={T} token {t}")


def test_many_tokens_degenerate_unions(api, c1, m7b):
    """Calls with more than 128 tokens whose union is tiny, empty, or a prefix that ends inside a tile."""
    cfg = c1.cfg
    n = cfg.n_loaded
    T = 256
    x = wl.x_tokens(cfg, 0, T, first_token=3)
    # five scattered slots shared by all tokens: one active weight tile, one K chunk of the down contraction
    shared = np.array([1, 17, 18, 400, n - 1], np.int32)
    y = _run(api, c1, 0, x, shared, None, len(shared), T, flags=api.SI_FLAG_SHARED_LIST)
    for t in (0, 100, 128, 255):
        assert_close(from_dev(y[t]), c1.oracle_y(0, x[t], shared), f"five shared slots, token {t}")
    # every list empty: y = x exactly (residual), y = 0 without it
    T = 200
    off = np.zeros(T + 1, np.int32)
    y = _run(api, c1, 0, x[:T], np.zeros(4, np.int32), off, n, T, flags=api.SI_FLAG_RESIDUAL)
    assert np.array_equal(from_dev(y), wl.bits_to_float64(x[:T], cfg.dtype))
    y = _run(api, c1, 0, x[:T], np.zeros(4, np.int32), off, n, T)
    assert not from_dev(y).any()
    # 129 tokens (the second CTA of the pair holds one token) over a prefix of 1000 slots of a 7B-shaped layer:
    # seven whole tiles fetched by tensor copies and a last tile of 104 real entries
    cfg7 = m7b.cfg
    T, k = 129, 1000
    x7 = wl.x_tokens(cfg7, 0, T, first_token=900)
    prefix = np.arange(k, dtype=np.int32)
    y = _run(api, m7b, 0, x7, prefix, None, k, T, flags=api.SI_FLAG_SHARED_LIST, y_dtype=torch.bfloat16)
    for t in (0, 127, 128):
        assert_close(from_dev(y[t]), m7b.oracle_y(0, x7[t], prefix), f"129 tokens, token {t}")


@pytest.mark.parametrize("T", [48, 100, 128])
def test_7b_up_to_128_tokens_cluster_split(api, m7b, T):
    """The widest token tiles of the one-CTA kernels (48, 112 and 128 columns of tensor memory per accumulator): K is
    split over a thread-block cluster and the partial accumulators are summed through distributed shared memory,
    whose staging area grows with the token count.  Own lists, residual, 16-bit output; run twice: bit-stable."""
    cfg = m7b.cfg
    k = cfg.k_active
    lists = wl.zipf_lists(cfg, 0, T, first_token=5)
    x = wl.x_tokens(cfg, 0, T, first_token=40)
    y = _run(api, m7b, 0, x, lists, None, k, T, flags=api.SI_FLAG_RESIDUAL, y_dtype=torch.bfloat16)
    for t in sorted({0, 15, 16, T // 2, T - 1}):
        ref = m7b.oracle_y(0, x[t], lists[t]) + wl.bits_to_float64(x[t], cfg.dtype)
        assert_close(from_dev(y[t]), ref, f"T={T} token {t}")
    y2 = _run(api, m7b, 0, x, lists, None, k, T, flags=api.SI_FLAG_RESIDUAL, y_dtype=torch.bfloat16)
    assert torch.equal(y, y2)
