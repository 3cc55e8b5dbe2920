"""Child of the launcher test: joins a gloo group with the environment the launcher gave it and writes what it saw."""
import os
import sys

import torch
import torch.distributed as dist

out_dir = sys.argv[1]
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
t = torch.tensor([float(rank + 1)])
dist.all_reduce(t, op=dist.ReduceOp.SUM)
with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
    f.write(f"{rank} {world} {os.environ['LOCAL_RANK']} {int(t.item())} {os.getpid()}\n")
dist.destroy_process_group()
