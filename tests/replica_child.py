"""Child of tests/test_replicas_gloo.py::test_ensure_ranks_starts_the_ranks_itself: runs as one rank under
torch.distributed.run, joins a gloo group, and lets rank 0 write what the group saw."""
import json
import sys

import torch
import torch.distributed as dist

from paper_2607_18081_b200 import replicas

if __name__ == "__main__":
    rank, world, local = replicas.rank_info()
    dist.init_process_group("gloo")
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t)
    mx = replicas.max_over_ranks(10.0 + rank)
    replicas.barrier()
    if rank == 0:
        with open(sys.argv[1], "w") as f:
            json.dump({"world": world, "sum": float(t.item()), "max_ms": mx, "argv": sys.argv[2:]}, f)
    dist.destroy_process_group()
