"""bench.py prints one JSON line with the agreed keys (run on the smallest configuration)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_json_line_has_the_agreed_keys():
    out = subprocess.run([sys.executable, "bench.py", "--workload", "c1", "--steps", "60",
                          "--warmup", "3", "--min-time", "0.2"], cwd=ROOT, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "clocks",
                "timing", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["metric"] == "simulated_worker_steps_per_sec" and d["unit"] == "worker-steps/s"
    assert d["n_gpus"] == 1 and d["steps"] == 60 and d["warmup"] == 3
    assert d["value"] > 0 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and "workload" in d["config"] and "model" not in d["config"]
    assert abs(d["value"] - 4 * 60 / (d["ms_per_step"] * 60 * 1e-3)) <= 0.01 * d["value"]
    assert d["gpu_launches"] > 0
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] == 4 * 32 * 64 * 4 + 4 * 32 * 4
    assert e["d2h_bytes_per_step"] == 16 and e["value"] != d["value"]
    r = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in r, key
    assert r["bound"] == "hbm" and r["unit"] == "GB/s"
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    # the timed region: repeated blocks of exactly `steps` iterations, the median reported
    t = d["timing"]
    assert t["blocks"] >= 2 and t["timed_s"] >= 0.2
    assert t["ms_per_step_min"] <= t["ms_per_step_median"] <= t["ms_per_step_max"]
    assert t["ms_per_step_median"] == d["ms_per_step"] and "olsgd_run" in t["path"]
    assert d["graph_replays"] > 0 and "replay" in t["path"]
    assert e["blocks"] >= 2 and e["ms_per_step_min"] <= e["ms_per_step"] <= e["ms_per_step_max"]
    # no hidden layers: the roofline entry describes the model's own kernels, rows read once
    assert r["kernel"] == "output_layer"
    assert r["algorithmic_bytes_per_launch"] >= 4 * 32 * 64 * 4
    # the update and anchor kernels by themselves, at config 5's two quoted points
    alone = [k for k in r["kernels"] if k["kernel"] in ("fused_update_kernel", "worker_mean_anchor_kernel")]
    assert len(alone) == 4
    for k in alone:
        assert k["gbs"] > 0 and 0 < k["frac_of_measured"] < 1.5 and 0 < k["frac_of_8000"] < 1.2
        assert "config 5" in k["workload"]
    # the oracle on all cores and on one core, thread counts stated
    assert c["one_core"]["cores"] == 1 and c["one_core"]["value"] > 0 and "BLAS threads" in c["sample"]


def test_bench_mlp_line_reports_every_gemm_launch():
    out = subprocess.run([sys.executable, "bench.py", "--workload", "c3", "--steps", "20",
                          "--warmup", "3", "--min-time", "0.3", "--no-kernel-points"], cwd=ROOT,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][0])
    r = d["roofline"]
    assert r["kernel"] == "wgrad_update" and 0.3 < r["frac"] < 1.3
    gemms = [k for k in r["kernels"] if k["kernel"].startswith("gemm_tc_kernel")]
    assert len(gemms) == 3            # two forward GEMMs, one input-gradient GEMM
    for k in gemms:
        assert k["us"] > 0 and k["tflops"] > 0 and 0 < k["frac_of_bound"] <= 1.2
        assert k["bound"] in ("hbm", "tensor") and 0 < k["frac_of_bf16_peak"] < 1
    assert d["graph_replays"] > 0 and d["timing"]["blocks"] >= 2
    assert d["e2e"]["h2d_bytes_per_step"] == 16 * 128 * 3072 * 2 + 16 * 128 * 4
