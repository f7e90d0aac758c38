"""Rank body for test_dist_replicas.py::test_launch_ranks...: joins a gloo group with the environment the
launcher set and leaves one file per rank."""
import os
import sys

import torch
import torch.distributed as dist

out_dir = sys.argv[1]
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
t = torch.tensor([rank + 1.0])
dist.all_reduce(t)
with open(os.path.join(out_dir, "rank%d.txt" % rank), "w") as f:
    f.write("%d %d %d %s %.0f\n" % (rank, world, int(os.environ["LOCAL_RANK"]), os.environ["MASTER_ADDR"], float(t[0])))
dist.barrier()
dist.destroy_process_group()
