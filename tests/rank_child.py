"""Child process of the rank-launcher test: joins a gloo group from the environment the launcher sets, sums
rank + 1 over the ranks, and rank 0 prints one JSON line, the way bench.py does."""
import json
import os
import sys

import torch
import torch.distributed as dist

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo")      # env:// rendezvous
t = torch.tensor([float(rank + 1)])
dist.all_reduce(t)
slowest = torch.tensor([10.0 + rank])
dist.all_reduce(slowest, op=dist.ReduceOp.MAX)
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "sum": float(t[0]), "max_ms": float(slowest[0]), "argv": sys.argv[1:]}), flush=True)
dist.destroy_process_group()
