"""Worker of tests/test_multi_rank.py: one gloo rank on CPU exercising bench.py's cross-rank logic."""
import json
import os
import sys

import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# every rank is an independent replica with its own timings; rank 1 is the slow one
mine = [10.0 + rank, 100.0 + 7 * rank, 111.0 + 8 * rank]
red = bench.reduce_max_over_ranks(mine, dist, torch.device("cpu"))
dist.barrier()
if rank == 0:
    print(json.dumps({"reduced": red, "world": world,
                      "value": bench.whole_job_rate(16 * 128, world, red[1] * 1e-3)}))
dist.destroy_process_group()
