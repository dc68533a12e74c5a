"""World-size-2 check of the replica plumbing on CPU (gloo): disjoint token ranges, the max over
ranks of the timed region, and the whole-job throughput formula."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_18081_b200 import replicas, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.rank_info() == (rank, world, rank)
    first, last = replicas.token_range(rank, world, 5)
    cfg = wl.CONFIGS["c1"]
    ids, sor = wl.loaded_ids(cfg, 0)
    lists = wl.zipf_lists(cfg, 0, last - first, slot_of_rank=sor, first_token=first)
    replicas.barrier()
    mine_ms = 10.0 + 7.0 * rank                      # rank 1 is the slow one
    mx = replicas.max_over_ranks(mine_ms)
    out[rank] = (first, last, int(lists.sum()), mx)
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert (r0[0], r0[1]) == (0, 5) and (r1[0], r1[1]) == (5, 10)       # disjoint, contiguous
    assert r0[2] != r1[2]                                               # different tokens -> different lists
    assert r0[3] == r1[3] == 17.0                                       # both see the slow rank's time
    assert replicas.aggregate_throughput(128, 2, 17.0) == 2 * 128 / 0.017


def test_single_process_defaults():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.token_range(0, 1, 128) == (0, 128)
