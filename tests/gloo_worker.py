"""Run under torchrun with the gloo backend by test_bench_reference_arm.py: checks the
max-over-ranks reduction bench.py uses for its timings and the replica seeding rule."""
import os
import sys

import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
got = bench.max_over_ranks(10.0 + rank, world, "cpu")
assert got == 10.0 + world - 1, got
dist.barrier()
dist.destroy_process_group()
if rank == 0:
    print("GLOO_OK", world)
