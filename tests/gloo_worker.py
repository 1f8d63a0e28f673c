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
# the record a multi-GPU run adds for the job whose WORKERS are sharded over the ranks: built
# from the slowest rank's time, the same on every rank
import json  # noqa: E402
import synth_inputs as si  # noqa: E402
c = si.CONFIGS["c3"]
ms = bench.max_over_ranks(5.0 + rank, world, "cpu")
rec = bench.sharded_summary(c, bench.n_params(c), world, ms, 20)
assert rec["workers_per_gpu"] * world == c["m"] and rec["n_gpus"] == world
assert rec["value"] == round(c["m"] * 20 / ((5.0 + world - 1) * 1e-3), 1)
dist.barrier()
dist.destroy_process_group()
if rank == 0:
    print("GLOO_OK", world)
    print("SHARDED " + json.dumps(rec))
