"""Multi-GPU plumbing: independent replicas, no data-path collective.

The selective-FFN path is a one-GPU path.  With N GPUs every rank holds its own copy of the
neuron store and decodes its own tokens (weak scaling); the only communication is the barrier
around the timed region and the max-over-ranks of the measured time.  Works with any
torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, world_size, local_rank) from the torchrun environment (1-process defaults)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def token_range(rank: int, world: int, tokens_per_rank: int):
    """Weak scaling: rank r decodes tokens [r * tokens_per_rank, (r + 1) * tokens_per_rank)."""
    if not 0 <= rank < world or tokens_per_rank < 0:
        raise ValueError("bad rank / world / tokens")
    first = rank * tokens_per_rank
    return first, first + tokens_per_rank


def max_over_ranks(value_ms: float, device=None) -> float:
    """Max of a per-rank time over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value_ms)
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: int, world: int, max_ms: float) -> float:
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return world * units_per_rank / (max_ms * 1e-3)


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def launch_command(n_ranks: int, script: str, argv, port: int | None = None):
    """Command line that starts `script argv...` as n_ranks processes of one node, one per GPU, the way
    the benchmark contract launches a multi-GPU run (torch.distributed.run, rendezvous on 127.0.0.1)."""
    import socket
    import sys
    if n_ranks < 1:
        raise ValueError("n_ranks must be positive")
    if port is None:
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script, *[str(a) for a in argv]]


def ensure_ranks(n_ranks: int, script: str, argv, env=None):
    """If n_ranks > 1 and this process was not started by a launcher (no WORLD_SIZE in the environment),
    start the ranks and return their exit code; otherwise return None and the caller carries on as the
    rank it is.  NCCL's communicator set-up lines are left on for the ranks (stderr) unless the caller's
    environment says otherwise, so a scaling run shows what transport it ran on."""
    import subprocess
    if n_ranks <= 1 or "WORLD_SIZE" in os.environ:
        return None
    child_env = dict(os.environ if env is None else env)
    child_env.setdefault("NCCL_DEBUG", "INFO")
    child_env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    return subprocess.call(launch_command(n_ranks, script, argv), env=child_env)
