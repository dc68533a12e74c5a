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


def test_ensure_ranks_starts_the_ranks_itself(tmp_path):
    """`bench.py --gpus N` without a launcher: the process starts its own N ranks (here 2 gloo ranks on
    CPU running a small child script) and hands their exit code back; inside a rank nothing is started."""
    import json
    import subprocess
    import sys
    cmd = replicas.launch_command(3, "x.py", ["--gpus", 3], port=1234)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=3" in cmd and cmd[-3:] == ["x.py", "--gpus", "3"] and "127.0.0.1" in cmd and "1234" in cmd
    out = tmp_path / "ranks.json"
    child = os.path.join(os.path.dirname(os.path.abspath(__file__)), "replica_child.py")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    env["PYTHONPATH"] = root + os.pathsep + env.get("PYTHONPATH", "")
    saved = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        assert replicas.ensure_ranks(1, child, [str(out)], env=env) is None          # one rank: nothing to start
        rc = replicas.ensure_ranks(2, child, [str(out), "--flag"], env=env)
        assert rc == 0
        got = json.loads(out.read_text())
        assert got == {"world": 2, "sum": 3.0, "max_ms": 11.0, "argv": ["--flag"]}
        os.environ["WORLD_SIZE"] = "2"                                                # already a rank: nothing is started
        assert replicas.ensure_ranks(2, child, [str(out)], env=env) is None
    finally:
        os.environ.pop("WORLD_SIZE", None)
        os.environ.update(saved)
