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
