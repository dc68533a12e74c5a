"""GPU parity of the neuron-sharded path on one GPU: si_shard_lists bit for bit against the oracle,
and P shares of one layer evaluated one after the other (each with its own store over its local
slots), their fp32 partial outputs added by si_shard_reduce in rank order, against the float64 oracle
of the whole layer.  Nothing here waits on another rank: the shares run as ordinary launches in one
stream."""
import numpy as np
import pytest
import torch

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import workloads as wl
from tests.gpu_utils import assert_close, from_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    from paper_2607_18081_b200 import api as _api
    return _api


def _status():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def _shard_lists(api, lists, rank, world, csr):
    n_lists = len(lists)
    if csr:
        flat = np.concatenate(lists).astype(np.int32) if n_lists else np.zeros(0, np.int32)
        off = np.zeros(n_lists + 1, dtype=np.int32)
        off[1:] = np.cumsum([len(l) for l in lists])
        idx = torch.from_numpy(np.concatenate([flat, np.zeros(4, np.int32)])).cuda()
        offsets, k_fixed = torch.from_numpy(off).cuda(), 0
    else:
        idx = torch.from_numpy(np.ascontiguousarray(np.stack(lists), dtype=np.int32)).cuda()
        offsets, k_fixed = None, len(lists[0])
    idx_out = torch.full((idx.numel() + 4,), -9, dtype=torch.int32, device="cuda")
    offsets_out = torch.full((n_lists + 1,), -9, dtype=torch.int32, device="cuda")
    ws = torch.empty((n_lists + 64) * 4, dtype=torch.uint8, device="cuda")
    st = _status()
    api.si_shard_lists(idx, offsets, k_fixed, n_lists, rank, world, idx_out, offsets_out, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    return idx_out.cpu().numpy(), offsets_out.cpu().numpy()


@pytest.mark.parametrize("world", [1, 2, 3, 7])
def test_shard_lists_bit_exact(api, world):
    g = np.random.default_rng(40 + world)
    n = 5000
    # ragged lists, empty ones among them, more lists than one scan round holds, one longer than a block round
    lens = [0, 1, 2, 255, 256, 257, 1300, n] + [int(v) for v in g.integers(0, 600, size=300)]
    lists = [np.sort(g.permutation(n)[:k]).astype(np.int32) for k in lens]
    for rank in range(world):
        got, off = _shard_lists(api, lists, rank, world, csr=True)
        want = so.shard_lists(lists, rank, world)
        assert off[0] == 0 and np.array_equal(np.diff(off), [len(w) for w in want])
        for t, w in enumerate(want):
            assert np.array_equal(got[off[t]:off[t + 1]], w), (world, rank, t)
    # fixed-length lists
    fixed = [np.sort(g.permutation(n)[:777]).astype(np.int32) for _ in range(5)]
    for rank in range(world):
        got, off = _shard_lists(api, fixed, rank, world, csr=False)
        want = so.shard_lists(fixed, rank, world)
        for t, w in enumerate(want):
            assert np.array_equal(got[off[t]:off[t + 1]], w)


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_layer_matches_whole_layer_oracle(api, world):
    from paper_2607_18081_b200 import sharded
    cfg = wl.Config("shardcase", 31, 1024, 1500, 1, "bf16", 60, 25, 8)
    wg, wu, wd = wl.layer_weights(cfg, 0)
    ids, sor = wl.loaded_ids(cfg, 0)
    d, k = cfg.d_model, cfg.k_active
    ranks = []
    for r in range(world):
        f = sharded.ShardedFFN(1, d, cfg.d_ff, cfg.n_loaded, cfg.n_base, cfg.dtype, r, world)
        f.load(0, to_dev(wg, cfg.dtype), to_dev(wu, cfg.dtype), to_dev(wd, cfg.dtype), ids)
        ranks.append(f)
    assert sum(f.plans[0].local_loaded for f in ranks) == cfg.n_loaded
    st = _status()
    for T in (1, 6, 40):
        lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=sor)
        x = wl.x_tokens(cfg, 0, T)
        xd = to_dev(x, cfg.dtype)
        idx = torch.from_numpy(lists).cuda()
        parts, total_local = [], 0
        for f in ranks:
            il, ol, k_cap = f.local_lists(0, idx, None, k, T, st)
            total_local += int(ol[-1].item())
            y32 = torch.full((T, d), 5.0, dtype=torch.float32, device="cuda")
            ws = f.store.workspace(T, k_cap, 1)
            f.forward_partial(0, xd, T, il, ol, k_cap, y32, ws, st)
            parts.append(y32)
        assert total_local == lists.size                         # every entry on exactly one rank
        y = torch.full((T, d), 3.0, dtype=torch.bfloat16, device="cuda")
        sharded.combine(parts, xd, T, d, y, api.SI_FLAG_RESIDUAL, cfg.dtype)
        y32 = torch.empty((T, d), dtype=torch.float32, device="cuda")
        sharded.combine(parts, None, T, d, y32, 0, cfg.dtype)
        torch.cuda.synchronize()
        assert st.item() == 0, api.strerror(int(st.item()))
        for t in range(0, T, 1 if T <= 8 else 9):
            ref = so.ffn(wg, wu, wd, x[t], ids[lists[t]], dtype=cfg.dtype, threads=so.host_threads())
            assert_close(from_dev(y32[t]), ref, f"world={world} T={T} token {t}")
            assert_close(from_dev(y[t]), ref + wl.bits_to_float64(x[t], cfg.dtype), f"world={world} T={T} token {t} +x")
        # the rank-order sum is what the kernel must produce, bit for bit
        acc = parts[0].clone()
        for p in parts[1:]:
            acc += p
        assert torch.equal(acc, y32)


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_decode_with_the_allreduce_inside_the_kernel(api, world):
    """Batch-1 decode of a sharded layer with the all-reduce inside the kernel that finishes the down projection.  All
    ranks of the group share this GPU, so they run as ONE launch over all ranks' data (their blocks wait on one
    another).  Every rank's output must be the same bits, equal to the rank-order sum of the ranks' partial outputs
    that the two-kernel path (partial output, then si_shard_reduce) gives, and within tolerance of the oracle of the
    whole layer; three calls in a row reuse the receive areas and the delivery marks."""
    from paper_2607_18081_b200 import sharded
    cfg = wl.Config("shardcase", 31, 1024, 1500, 1, "bf16", 60, 25, 8)
    wg, wu, wd = wl.layer_weights(cfg, 0)
    ids, sor = wl.loaded_ids(cfg, 0)
    d, k = cfg.d_model, cfg.k_active
    ranks = []
    for r in range(world):
        f = sharded.ShardedFFN(1, d, cfg.d_ff, cfg.n_loaded, cfg.n_base, cfg.dtype, r, world)
        f.load(0, to_dev(wg, cfg.dtype), to_dev(wu, cfg.dtype), to_dev(wd, cfg.dtype), ids)
        ranks.append(f)
    recv = [torch.zeros(2, world, d, dtype=torch.float32, device="cuda") for _ in range(world)]
    marks = [torch.zeros(world, d // 32, dtype=torch.int32, device="cuda") for _ in range(world)]
    st = _status()
    lists = wl.zipf_lists(cfg, 0, 3, slot_of_rank=sor)
    x = wl.x_tokens(cfg, 0, 3)
    for call, flags in enumerate((0, api.SI_FLAG_RESIDUAL, 0)):
        xd = to_dev(x[call], cfg.dtype)
        idx = torch.from_numpy(lists[call:call + 1]).cuda()
        local, parts, wss = [], [], []
        for f in ranks:
            il, ol, k_cap = f.local_lists(0, idx, None, k, 1, st)
            n_local = int(ol[1].item())
            local.append((il, n_local))
            ws = f.store.workspace(1, max(n_local, 1), 1)
            wss.append(ws)
            y32 = torch.empty(1, d, dtype=torch.float32, device="cuda")
            api.si_ffn_forward(f.store.handle, 0, xd, 1, il, None, n_local, y32, api.SI_FLAG_SIMPLE_KERNELS, ws, st)
            parts.append(y32)
        want = torch.empty(1, d, dtype=torch.float32, device="cuda")
        sharded.combine(parts, xd if flags else None, 1, d, want, flags, cfg.dtype)
        ys = [torch.full((d,), 7.0, dtype=torch.float32, device="cuda") for _ in range(world)]
        api.si_debug_ffn_forward_sharded_group([f.store.handle for f in ranks], 0, world, 0, [xd] * world, [il for il, _ in local],
                                               [n for _, n in local], ys, flags, recv, marks, call + 1, wss, st)
        torch.cuda.synchronize()
        assert st.item() == 0, api.strerror(int(st.item()))
        for r in range(world):
            assert torch.equal(ys[r], want[0]), f"call {call} rank {r}"
        ref = so.ffn(wg, wu, wd, x[call], ids[lists[call]], dtype=cfg.dtype, threads=so.host_threads())
        if flags:
            ref = ref + wl.bits_to_float64(x[call], cfg.dtype)
        assert_close(from_dev(ys[0]), ref, f"call {call}")
    # a rank that never delivers: the others' wait runs out, the status says so, the launch returns
    st.zero_()
    xd = to_dev(x[0], cfg.dtype)
    il, n_local = local[0]
    y0 = torch.empty(d, dtype=torch.float32, device="cuda")
    api.si_debug_ffn_forward_sharded_group([ranks[0].store.handle], 0, world, 0, [xd], [il], [n_local], [y0], 0, recv, marks, 4, [wss[0]],
                                           st, wait_cycles=2_000_000)
    torch.cuda.synchronize()
    assert st.item() == api.SI_ERR_TIMEOUT
