"""Run under torchrun with the gloo backend (CPU): checks bench.py's multi-rank timing reduction."""
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.reduce_max_ms(10.0 + 5.0 * rank, world)           # slowest rank decides
assert ms == 10.0 + 5.0 * (world - 1), ms
tops = bench.whole_job_tops(1e12, world, ms)                   # every rank does 1 Tera-op per step
assert abs(tops - world * 1e12 / (ms * 1e-3) / 1e12) < 1e-9
dist.barrier()
if rank == 0:
    print(f"GLOO_OK world={world} ms={ms}")
dist.destroy_process_group()
