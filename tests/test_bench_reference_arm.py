"""bench.py --impl reference (the CPU oracle as the reference arm) on CPU, single
process and under torchrun with two ranks: one JSON line, printed by rank 0 only."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _json_lines(out):
    return [json.loads(l) for l in out.splitlines() if l.startswith("{")]


def test_reference_arm_single_process():
    out = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--workload", "c1",
                          "--steps", "5", "--warmup", "3"], cwd=ROOT, capture_output=True,
                         text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = _json_lines(out.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["metric"] == "simulated_worker_steps_per_sec"
    assert d["unit"] == "worker-steps/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 5 and d["warmup"] == 3
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}


def test_reference_arm_two_ranks_rank0_prints():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29517", "bench.py", "--impl",
           "reference", "--workload", "c1", "--gpus", "2", "--steps", "4", "--warmup", "3"]
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = _json_lines(out.stdout)
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert "sharded" not in lines[0]      # the oracle arm runs on rank 0 alone: nothing is sharded


def test_max_over_ranks_with_two_gloo_ranks():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29518",
           os.path.join("tests", "gloo_worker.py")]
    out = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "GLOO_OK 2" in out.stdout
    # shape of the `sharded` record that bench.py --gpus N (N > 1) adds to its line
    rec = json.loads([l for l in out.stdout.splitlines() if l.startswith("SHARDED ")][0][8:])
    assert set(rec) >= {"value", "unit", "ms_per_step", "steps", "scaling", "workers_per_gpu", "m",
                        "n_gpus", "allreduce_bytes_per_period", "collective"}
    assert rec["unit"] == "worker-steps/s" and rec["scaling"] == "strong" and rec["n_gpus"] == 2
    assert rec["workers_per_gpu"] == 8 and rec["allreduce_bytes_per_period"] == 4 * 4206602
    assert rec["ms_per_step"] == 0.3          # the slower rank's 6 ms over 20 steps
