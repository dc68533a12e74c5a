"""World-size-2 check of the neuron-sharded path's host logic on CPU (gloo): the slot partition of
ShardPlan, and that partial outputs over the ranks' shares, all-reduced, give the full selective FFN.
The partial outputs here come from the oracle (no GPU in this test); the collective is the real one."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import selectinfer_oracle as so
from paper_2607_18081_b200 import sharded, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = wl.CONFIGS["c1"]
    wg, wu, wd = wl.layer_weights(cfg, 0)
    ids, sor = wl.loaded_ids(cfg, 0)
    plan = sharded.ShardPlan(cfg.n_loaded, cfg.n_base, rank, world)
    my_ids = plan.local_ids(ids)
    assert len(my_ids) == plan.local_loaded
    assert np.array_equal(my_ids, ids[so.shard_slots(cfg.n_loaded, rank, world)])
    assert plan.local_base == len([s for s in range(cfg.n_base) if s % world == rank])
    T = 3
    lists = wl.zipf_lists(cfg, 0, T, slot_of_rank=sor)
    x = wl.x_tokens(cfg, 0, T)
    mine = so.shard_lists(lists, rank, world)
    y = np.stack([so.ffn(wg, wu, wd, x[t], my_ids[mine[t]], dtype=cfg.dtype) for t in range(T)])
    yt = torch.from_numpy(y)
    dist.all_reduce(yt)                                           # the one collective of the path
    full = np.stack([so.ffn(wg, wu, wd, x[t], ids[lists[t]], dtype=cfg.dtype) for t in range(T)])
    out[rank] = (float(np.abs(yt.numpy() - full).max()), float(np.abs(full).max()), int(sum(len(m) for m in mine)),
                 int(lists.size))
    dist.destroy_process_group()


def test_two_neuron_shards_over_gloo():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    for err, scale, _, _ in (r0, r1):
        assert err <= 1e-12 * scale                               # float64 partial sums, reassociated once
    assert r0[2] + r1[2] == r0[3]                                 # every list entry lives on exactly one rank
    assert r0[2] > 0 and r1[2] > 0


def test_shard_plan_counts():
    for n, nb, world in ((10, 4, 3), (7705, 3302, 8), (5, 5, 8), (0, 0, 2)):
        plans = [sharded.ShardPlan(n, nb, r, world) for r in range(world)]
        assert sum(p.local_loaded for p in plans) == n
        assert sum(p.local_base for p in plans) == min(nb, n)
        for p in plans:
            assert p.local_loaded == len(so.shard_slots(n, p.rank, world))
            assert np.array_equal(p.global_slot(np.arange(p.local_loaded)), so.shard_slots(n, p.rank, world))
