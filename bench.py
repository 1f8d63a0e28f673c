#!/usr/bin/env python
"""Benchmark of the Overlap-Local-SGD hot path: simulated worker-steps per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c1|c5]
                    [--impl ours|reference]

One "step" is one iteration k -> k+1 for all m workers: minibatch indices,
gather, forward, loss, backward, fused update (+ pull-back on sync steps) and,
every tau steps, the anchor refresh on the side stream.  Prints one JSON line.

With N > 1 (launched by torchrun, one rank per GPU) every rank runs an
independent replica of the whole m-worker job on its own seed; there is no
collective on the data path.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "simulated_worker_steps_per_sec"
UNIT = "worker-steps/s"
L2_BYTES = 126 * 2 ** 20
MAX_BLOCKS = 20000         # upper bound on repeated timed blocks


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


# ------------------------------------------------------------------ inputs

def make_inputs(name, seed, class_table=None):
    c = si.CONFIGS[name]
    if c["kind"] == "linreg":
        X, y, _ = si.linreg_data(seed, c["m"], c["n"], c["dims"][0])
    else:
        X, y = si.mixture_data(seed, c["m"], c["n"], c["dims"][0], class_table)
    x0 = si.model_init(seed, c["kind"], c["dims"])
    return X, y, x0


def n_params(c):
    d = c["dims"]
    if c["kind"] == "linreg":
        return d[0]
    return sum(d[l + 1] * d[l] + d[l + 1] for l in range(len(d) - 1))


# ------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def wait_first_sample(self, limit_s=5.0):
        """nvidia-smi holds driver locks while it starts up, which can stall kernel launches for
        tens of milliseconds: the timed region begins only after its first sample has arrived."""
        t0 = time.time()
        while self.proc is not None and not self.lines and time.time() - t0 < limit_s:
            time.sleep(0.01)

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [t.strip() for t in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=float(np.median(sm)) if sm else None,
                    sm_max_mhz=float(np.max(mx)) if mx else None, reasons=sorted(reasons),
                    samples=len(sm))


# ------------------------------------------------------------------ roofline accounting

def git_blob_id(path):
    """The id git gives a file's content (sha1 of the header "blob <size>" + NUL + bytes)."""
    import hashlib
    with open(path, "rb") as f:
        data = f.read()
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


CSRC = os.path.join(ROOT, "paper_2002_09539_b200", "csrc")

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch from the ncu capture
# summarised in profiles/, keyed by (workload, gemm mode, kernel class): (ordinary step, sync
# step), the kernel's source file and that file's git blob id when the counters were taken.
# When the file has changed since, the entry no longer describes the kernel and `traffic`
# is reported as null.
NCU_TRAFFIC = {
    # profiles/wgrad_update_fused_c3_mlp.txt
    ("c3", 1, "wgrad_update"): (1179.9e6, 1294.8e6, "tc_wgrad.cu", "3aed0e701941734c2348052d213ea589fb019b40"),
    # profiles/wgrad_update_fused_c4_mlp.txt
    ("c4", 1, "wgrad_update"): (1787.0e6, 1897.0e6, "tc_wgrad.cu", "3aed0e701941734c2348052d213ea589fb019b40"),
}


def ncu_traffic(name, mode, kernel_class, sync_fraction):
    t = NCU_TRAFFIC.get((name, mode, kernel_class))
    if t is None:
        return None
    plain, sync, source, blob = t
    try:
        if git_blob_id(os.path.join(CSRC, source)) != blob:
            return None
    except OSError:
        return None
    return int((1.0 - sync_fraction) * plain + sync_fraction * sync)


def layer_is_fused(c, p):
    """Does the weight-gradient GEMM of parameter layer p apply the update in its epilogue?"""
    d = c["dims"]
    return (c.get("gemm_bf16") == 1 and p < len(d) - 2 and d[p + 1] % 128 == 0 and
            d[p] % 128 == 0 and c["batch"] % 64 == 0 and c["batch"] <= 128)


def fused_weight_count(c):
    d = c.get("dims", [])
    return sum(d[p + 1] * d[p] for p in range(len(d) - 2) if layer_is_fused(c, p))


def algorithmic_bytes(c, kernel_class, P, sync_fraction):
    """Algorithmic HBM bytes of ONE launch of the given kernel class (averaged over
    sync and ordinary steps for the update kernel)."""
    m = c["m"]
    mom = c["mu"] != 0.0
    shadow = 2 if c.get("gemm_bf16") else 0
    fused = fused_weight_count(c)
    if kernel_class == "wgrad_update":
        # one launch covers all fused layers: x read+write, u read+write, bf16 shadow write
        # per parameter per worker, the anchor once on sync steps, the bf16 operands once
        if not fused:
            return None
        d, B = c["dims"], c["batch"]
        layers = [p for p in range(len(d) - 2) if layer_is_fused(c, p)]
        per = (16 if mom else 8) + 2
        operands = sum(m * B * 2 * (d[p + 1] + d[p]) for p in layers)
        # sync steps: the anchor read once, and (worker sum formed in the launch) one row of
        # partial sums written per slice
        slices = c.get("sum_slices", 0)
        return m * fused * per + sync_fraction * 4 * (1 + slices) * fused + operands
    if kernel_class == "update":
        # sync steps: the anchor read once, and (worker sum formed in the launch, long rows
        # only) one row of partial sums written per slice
        per = (20 if mom else 12) + shadow
        rest = P - fused
        return m * rest * per + sync_fraction * 4 * (1 + c.get("update_sum_slices", 0)) * rest
    if kernel_class == "anchor":
        return 4 * m * P + (16 if c["beta"] != 0.0 else 4) * P
    if kernel_class == "output_layer" and c.get("kind") in ("softmax", "linreg"):
        # the kernels of a model without hidden layers (forward + loss, weight gradient with the
        # update applied on the spot): the step's minibatch rows ONCE, the parameters read by
        # the forward pass, read and written by the update (with the momentum buffer, if any),
        # the anchor once on sync steps
        rows = m * c["batch"] * c["dims"][0] * 4
        return rows + m * P * (4 + 8 + (8 if mom else 0)) + sync_fraction * 4 * P
    return None


def gemm_rooflines(c, layers_prof, n_steps, peaks):
    """Per tcgen05 GEMM launch of the MLP path: duration, TFLOP/s and the fraction of its bound,
    min(bf16 peak, arithmetic intensity x HBM bandwidth), from the per-layer device profile."""
    if c.get("kind") != "mlp" or not c.get("gemm_bf16"):
        return []
    d, m, B = c["dims"], c["m"], c["batch"]
    L = len(d) - 1
    peak_flops = peaks["bf16_tflops"] * 1e12
    hbm = peaks["hbm_gbs"] * 1e9
    out = []

    def entry(name, cls, tag, flops, nbytes):
        launches, ms = layers_prof[cls][tag]
        if launches <= 0:
            return
        us = ms * 1e3 / launches
        bound_s = max(flops / peak_flops, nbytes / hbm)
        out.append(dict(kernel=name, launches_per_step=round(launches / n_steps, 3), us=round(us, 2),
                        tflops=round(flops / (us * 1e-6) / 1e12, 1),
                        frac_of_bf16_peak=round(flops / (us * 1e-6) / peak_flops, 4),
                        flop_per_byte=round(flops / nbytes, 1), bound_us=round(bound_s * 1e6, 2),
                        bound="hbm" if nbytes / hbm > flops / peak_flops else "tensor",
                        frac_of_bound=round(bound_s * 1e6 / us, 4)))

    for l in range(1, L):
        # forward: W_l [d_l][d_{l-1}] bf16 read once, the batch operand read, H_l written in
        # both layouts
        flops = 2.0 * m * B * d[l] * d[l - 1]
        nbytes = m * (2 * d[l] * d[l - 1] + 2 * B * d[l - 1] + 4 * B * d[l])
        entry("gemm_tc_kernel forward, layer %d (%dx%d, batch %d)" % (l, d[l], d[l - 1], B),
              "forward", l, flops, nbytes)
    for l in range(1, L - 1):
        # input gradient of hidden layer l: W_{l+1} read in place (bf16 shadow), dA_{l+1} read,
        # the ReLU mask read, dA_l written in both layouts
        flops = 2.0 * m * B * d[l] * d[l + 1]
        nbytes = m * (2 * d[l + 1] * d[l] + 2 * B * d[l + 1] + 2 * B * d[l] + 4 * B * d[l])
        entry("gemm_tc_kernel input gradient, layer %d (%dx%d, batch %d)" % (l, d[l], d[l + 1], B),
              "backward", l, flops, nbytes)
    return out


def worker_sum_slices(m):
    """Rows of partial sums the library forms the worker sum in (a function of m alone)."""
    return 4 if m >= 64 else 2 if m >= 8 else 1


def flat_point(P, m, K, W, peaks):
    """Config 5 at one (P, m): a flat parameter vector with external gradients.  The whole
    iteration is timed as the library runs it by default (on long rows the sync step's update
    launch also forms the worker sums, and the anchor refresh starts from those few rows) and
    with the worker sum left to the worker-mean kernel; the kernels are timed one by one with
    the two streams serialised.  Returns the point's record."""
    import torch
    from paper_2002_09539_b200 import OverlapLocalSGD
    c = si.CONFIGS["c5"]
    tau = c["tau"]
    x0 = torch.randn(P, device="cuda")
    g = torch.randn((m, P), device="cuda") * c["grad_std"]
    kw = dict(m=m, tau=tau, gamma=c["gamma"], alpha=c["alpha"], beta=c["beta"], mu=c["mu"],
              flat_P=P, x0=x0)

    def steps(opt, count):
        for _ in range(count):
            opt.local_step_with_grads(g)
            if opt.iteration % tau == 0:
                opt.period_sync()

    def timed(fusion):
        opt = OverlapLocalSGD("flat", **kw)
        opt.set_anchor_fusion(fusion)
        steps(opt, W)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = opt.launch_count
        e0.record()
        steps(opt, K)
        opt.main.wait_stream(opt.side)
        e1.record()
        torch.cuda.synchronize()
        ms, launches, summed = e0.elapsed_time(e1), opt.launch_count - n0, opt.summed_floats
        opt.profile_enable(True)
        steps(opt, K)
        prof = opt.profile_read()
        opt.profile_enable(False)
        opt.close()
        return ms, launches, summed, prof

    def per_kernel(fusion):
        # with the two streams serialised: under overlap the anchor kernel shares HBM with the
        # next period's update kernels and its event-bracketed duration measures that sharing
        opt = OverlapLocalSGD("flat", overlap=False, **kw)
        opt.set_anchor_fusion(fusion)
        steps(opt, W)
        opt.profile_enable(True)
        steps(opt, K)
        prof = opt.profile_read_layers()
        opt.profile_enable(False)
        opt.close()
        return {(cls, tag): (prof[cls][tag][1] / prof[cls][tag][0] if prof[cls][tag][0] else None)
                for cls in ("update", "anchor") for tag in (0, 1)}

    ms, launches, summed, prof_overlap = timed(True)
    ms_plain = timed(False)[0] if summed else ms
    ref = per_kernel(False)          # the stand-alone update kernel and the worker-mean kernel
    cc = dict(c, m=m)
    S = worker_sum_slices(m)
    mom_rows = 16 if c["beta"] != 0.0 else 4
    upd_b = algorithmic_bytes(cc, "update", P, 0)
    upd_sync_b = algorithmic_bytes(cc, "update", P, 1)
    anc_b = algorithmic_bytes(cc, "anchor", P, 0)
    n_sync = K // tau
    # one figure for the update kernel, as before: all its launches, sync steps included
    upd_ms = (ref[("update", 0)] * (K - n_sync) + ref[("update", 1)] * n_sync) / K
    upd_all_b = (upd_b * (K - n_sync) + upd_sync_b * n_sync) / K
    anc_ms = ref[("anchor", 0)]
    state_mb = (3 * m * P + 2 * P + m * P) * 4 / 1e6
    gbs = lambda nbytes, t_ms: round(nbytes / t_ms / 1e6, 1)
    frac = lambda nbytes, t_ms, peak: round(nbytes / t_ms / 1e6 / peak, 4)
    point = dict(
        P=P, m=m, worker_steps_per_s=round(m * K / (ms * 1e-3), 1),
        ms_per_step=round(ms / K, 4), gpu_launches=int(launches),
        worker_sum_in_update_launch=bool(summed),
        ms_per_step_worker_mean_kernel=round(ms_plain / K, 4),
        update_gbs=gbs(upd_all_b, upd_ms), anchor_gbs=gbs(anc_b, anc_ms),
        update_us=round(upd_ms * 1e3, 2), anchor_us=round(anc_ms * 1e3, 2),
        anchor_us_overlapped=round(prof_overlap["anchor"][1] * 1e3 /
                                   max(1, prof_overlap["anchor"][0]), 2),
        update_frac_measured=frac(upd_all_b, upd_ms, peaks["hbm_gbs"]),
        anchor_frac_measured=frac(anc_b, anc_ms, peaks["hbm_gbs"]),
        update_frac_8000=frac(upd_all_b, upd_ms, 8000.0),
        anchor_frac_8000=frac(anc_b, anc_ms, 8000.0),
        resident_mb=round(state_mb, 1), in_l2=bool(state_mb * 1e6 < L2_BYTES))
    if summed:
        fused = per_kernel(True)
        sum_b = upd_sync_b + 4 * S * P           # the sync-step launch also writes S rows of sums
        fin_b = (4 * S + mom_rows) * P           # and the refresh reads them, with z and v
        point.update(
            sum_slices=S,
            sync_update_sum_us=round(fused[("update", 1)] * 1e3, 2),
            sync_update_sum_gbs=gbs(sum_b, fused[("update", 1)]),
            sync_update_sum_frac_measured=frac(sum_b, fused[("update", 1)], peaks["hbm_gbs"]),
            sync_update_plain_us=round(ref[("update", 1)] * 1e3, 2),
            anchor_from_sums_us=round(fused[("anchor", 1)] * 1e3, 2),
            anchor_from_sums_gbs=gbs(fin_b, fused[("anchor", 1)]),
            anchor_from_sums_frac_measured=frac(fin_b, fused[("anchor", 1)], peaks["hbm_gbs"]),
            sync_bytes_saved_per_period=int(anc_b - fin_b - 4 * S * P))
    del g, x0
    torch.cuda.empty_cache()
    return point


def standalone_kernel_rooflines(peaks, steps=12, warmup=4):
    """The metric's second half: the stand-alone fused update kernel and the worker-mean/anchor
    kernel on config 5's 10M x 16 and 50M x 64 points, streams serialised, as HBM GB/s against
    the measured copy bandwidth and against 8 TB/s; and the two launches that replace them on
    sync steps (update with the worker sum inside, anchor refresh from the partial sums)."""
    out = []
    for P, m in ((10_000_000, 16), (50_000_000, 64)):
        pt = flat_point(P, m, steps, warmup, peaks)
        where = "config 5, P=%dM, m=%d, tau=4, momentum, streams serialised" % (P // 1_000_000, m)
        out.append(dict(kernel="fused_update_kernel", workload=where, us=pt["update_us"],
                        gbs=pt["update_gbs"], frac_of_measured=pt["update_frac_measured"],
                        frac_of_8000=pt["update_frac_8000"]))
        out.append(dict(kernel="worker_mean_anchor_kernel", workload=where, us=pt["anchor_us"],
                        gbs=pt["anchor_gbs"], frac_of_measured=pt["anchor_frac_measured"],
                        frac_of_8000=pt["anchor_frac_8000"]))
        if pt["worker_sum_in_update_launch"]:
            out.append(dict(kernel="fused_update_kernel<SUM> (sync steps)", workload=where,
                            us=pt["sync_update_sum_us"], gbs=pt["sync_update_sum_gbs"],
                            frac_of_measured=pt["sync_update_sum_frac_measured"],
                            us_without_the_sum=pt["sync_update_plain_us"]))
            out.append(dict(kernel="anchor_from_slices_kernel", workload=where,
                            us=pt["anchor_from_sums_us"], gbs=pt["anchor_from_sums_gbs"],
                            frac_of_measured=pt["anchor_from_sums_frac_measured"]))
    return out


# ------------------------------------------------------------------ our arm

def run_ours(args, rank, world):
    import torch
    import torch.distributed as dist
    from paper_2002_09539_b200 import OverlapLocalSGD, class_pairs
    from paper_2002_09539_b200.build import build

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    # everything below runs on one real stream (the library's main stream, the timing events,
    # torch's copies): olsgd_run can only capture its CUDA graph on a non-default stream
    torch.cuda.set_stream(torch.cuda.Stream())

    name = args.workload
    c = dict(si.CONFIGS[name])
    if c["gemm_bf16"] and args.gemm_mode:
        c["gemm_bf16"] = args.gemm_mode
    local_sgd = args.method != "overlap"
    if args.tau:
        c["tau"] = args.tau          # a study of the sync cost, not the configuration's own period
    if args.method == "sync_sgd":
        c["tau"] = 1                 # fully synchronous SGD = Eq. 2 with tau = 1
    seed = rank                      # every rank is an independent replica
    table = None
    if c.get("non_iid"):
        table = class_pairs(seed, c["m"], device="cpu").numpy()
    X, y, x0 = make_inputs(name, seed, table)
    P = n_params(c)
    Xd, yd = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
    opt = OverlapLocalSGD(c["kind"], m=c["m"], tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=seed, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=Xd, y=yd, local_sgd=local_sgd)
    if args.no_anchor_fusion:
        opt.set_anchor_fusion(False)
    m, K, W = c["m"], args.steps, args.warmup

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        opt.main.wait_stream(opt.side)
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    # ---- device-resident throughput
    # W warm-up steps as asked, then (still untimed) one run long enough for olsgd_run to
    # capture its block of iterations, so that the timed blocks replay it.  A timed block is
    # EXACTLY K steps between a barrier + synchronize on both sides; blocks are repeated until
    # MIN_TIMED_S have been timed, and the median block is reported.
    opt.run(W)
    block = opt.graph_block
    opt.run(K if block <= K <= 64 else 3 * block)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
    launches0, replays0 = opt.launch_count, opt.graph_replays
    times = [timed(lambda: opt.run(K))]
    launches = opt.launch_count - launches0
    # (the block times are maxima over the ranks, so every rank takes the same decision)
    while sum(times) < args.min_time * 1e3 and len(times) < MAX_BLOCKS:
        times.append(timed(lambda: opt.run(K)))
    replays = opt.graph_replays - replays0
    clocks = sampler.stop() if rank == 0 else None
    ms = float(np.median(times))
    value = world * m * K / (ms * 1e-3)
    per_block = replays // len(times)
    unit = c["tau"] if c["tau"] % 2 == 0 else 2 * c["tau"]
    glen = K // unit * unit if block <= K <= 64 else block      # what olsgd_run captures for this K
    timing = dict(blocks=len(times), timed_s=round(sum(times) * 1e-3, 3),
                  ms_per_step_median=round(ms / K, 4), ms_per_step_min=round(min(times) / K, 4),
                  ms_per_step_max=round(max(times) / K, 4),
                  path=("olsgd_run: %d replay(s) of the captured %d-iteration graph + %d plain "
                        "step(s) per timed block" % (per_block, glen, K - per_block * glen))
                  if per_block else "olsgd_run: plain launches (K is shorter than the captured block)")

    # ---- per-kernel-class device time (second pass, every launch bracketed by events)
    # (a refresh has run by now: summed_floats says whether any launch formed worker sums)
    anchor_fusion_on = opt.anchor_fusion and opt.summed_floats > 0
    KP = max(K, 2 * block)
    opt.profile_enable(True)
    opt.run(KP)
    layers_prof = opt.profile_read_layers()
    opt.profile_enable(False)
    prof = {k: (sum(t[0] for t in v), sum(t[1] for t in v)) for k, v in layers_prof.items()}
    busy = {k: v for k, v in prof.items() if v[0] > 0}
    total_ms = sum(v[1] for v in busy.values())
    dominant = max(busy, key=lambda k: busy[k][1])
    peaks = measured_peaks()
    n_sync = sum(1 for k in range(KP) if (k + 1) % c["tau"] == 0) if not local_sgd else 0
    if c["kind"] in ("softmax", "linreg"):
        # no hidden layers: the time is in the output-layer kernels (forward + loss, weight
        # gradient with the update), which together need the step's rows once
        roof_class = "output_layer"
        parts = [k for k in ("forward", "loss", "backward") if k in busy]
        avg_ms = sum(busy[k][1] / busy[k][0] for k in parts)
    else:
        # the HBM-bound kernel class that took the most device time
        ranked = sorted(busy, key=lambda k: -busy[k][1])
        roof_class = next((k for k in ranked if algorithmic_bytes(c, k, P, 0) is not None), None)
        avg_ms = busy[roof_class][1] / busy[roof_class][0] if roof_class else None
    if roof_class is not None:
        if anchor_fusion_on:
            c = dict(c, sum_slices=worker_sum_slices(c["m"]))
            if fused_weight_count(c) == 0 and opt.summed_floats > 0:
                c["update_sum_slices"] = c["sum_slices"]     # the stand-alone update kernel sums
        ab = algorithmic_bytes(c, roof_class, P, n_sync / KP)
        achieved = ab / (avg_ms * 1e-3) / 1e9
        traffic = ncu_traffic(name, c["gemm_bf16"], roof_class, n_sync / KP)
        roofline = dict(bound="hbm", kernel=roof_class, achieved=round(achieved, 1),
                        peak=peaks["hbm_gbs"], unit="GB/s", frac=round(achieved / peaks["hbm_gbs"], 4),
                        frac_of_8000=round(achieved / 8000.0, 4), traffic=traffic,
                        peak_source=peaks["source"], avg_launch_us=round(avg_ms * 1e3, 2),
                        algorithmic_bytes_per_launch=int(ab))
        if traffic:
            # the same launch by the DRAM counters of the ncu capture instead of the byte count
            roofline.update(achieved_by_traffic=round(traffic / (avg_ms * 1e-3) / 1e9, 1),
                            frac_by_traffic=round(traffic / (avg_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4))
    else:
        roofline = dict(bound="hbm", kernel=None, achieved=None, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=None, traffic=None, peak_source=peaks["source"])
    roofline.update(dominant_class=dominant,
                    class_share={k: round(v[1] / total_ms, 4) for k, v in busy.items()},
                    class_us_per_step={k: round(v[1] * 1e3 / KP, 2) for k, v in busy.items()},
                    kernels=[])
    if c["kind"] == "mlp" and c["gemm_bf16"]:
        # The tensor-core GEMMs one launch at a time: a second context with the library's
        # streams serialised (no anchor refresh, gather or output-layer kernel beside them),
        # so that the bracketed duration is the kernel's own; warm caches, as inside a step.
        ser = OverlapLocalSGD(c["kind"], m=c["m"], tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                              beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=seed, dims=c["dims"],
                              gemm_bf16=c["gemm_bf16"], x0=x0, X=Xd, y=yd, local_sgd=local_sgd,
                              overlap=False)
        ser.run(W)
        ser.profile_enable(True)
        ser.run(KP)
        ser_prof = ser.profile_read_layers()
        ser.profile_enable(False)
        ser.close()
        del ser
        roofline["kernels"] = gemm_rooflines(c, ser_prof, KP, peaks)
        # the weight-gradient/update launch on ordinary and on sync steps, from the same pass
        for tag, what in ((0, "ordinary step"), (1, "sync step: pull-back" +
                                                 (", worker sums" if anchor_fusion_on else ""))):
            launches_t, ms_t = ser_prof["wgrad_update"][tag]
            if launches_t > 0:
                cc = dict(c, sum_slices=worker_sum_slices(c["m"]) if anchor_fusion_on else 0)
                ab_t = algorithmic_bytes(cc, "wgrad_update", P, float(tag))
                us_t = ms_t * 1e3 / launches_t
                roofline["kernels"].append(dict(
                    kernel="wgrad_tc_kernel<FUSED%s>, %s" % (", SUM" if tag and anchor_fusion_on else "", what),
                    us=round(us_t, 2), gbs=round(ab_t / us_t / 1e3, 1),
                    frac_of_measured=round(ab_t / us_t / 1e3 / peaks["hbm_gbs"], 4),
                    frac_of_8000=round(ab_t / us_t / 1e3 / 8000.0, 4),
                    algorithmic_bytes_per_launch=int(ab_t)))
        roofline["kernels_note"] = ("GEMM launches timed with the library's streams serialised "
                                    "(each kernel alone on the GPU, warm caches)")

    # ---- end to end: host minibatches in, host losses out, through the C ABI
    pool = 4
    n, B, d0 = c["n"], c["batch"], c["dims"][0]
    rng = np.random.default_rng(seed + 77)
    Xh, yh = [], []
    # a model whose GEMM operands are bf16 takes its rows in bf16 (the host data set is kept
    # in the operand type; rounding to nearest even on the host gives the bits the device's
    # own rounding of fp32 rows gives), any other model in fp32
    host_dtype = torch.bfloat16 if c["gemm_bf16"] else torch.float32
    for _ in range(pool):
        idx = rng.integers(0, n, size=(m, B))
        Xh.append(torch.from_numpy(np.stack([X[i][idx[i]] for i in range(m)])).to(host_dtype).pin_memory())
        yh.append(torch.from_numpy(np.stack([y[i][idx[i]] for i in range(m)])).pin_memory())
    loss_h = torch.zeros((K, m), dtype=torch.float32).pin_memory()

    def e2e_steps(count):
        for t in range(count):
            opt.local_step_host(Xh[t % pool], yh[t % pool], loss_h[t % K])
            if (opt.iteration) % c["tau"] == 0 and not local_sgd:
                opt.period_sync()

    def e2e_block():
        # K steps from pinned host rows to host-visible losses, by the host's clock
        barrier()
        t0 = time.perf_counter()
        e2e_steps(K)
        opt.join()                      # host sees the last losses here
        t1 = time.perf_counter()
        return max_over_ranks((t1 - t0) * 1e3, world, "cuda")

    e2e_steps(W)
    opt.join()
    e2e_times = [e2e_block()]
    while sum(e2e_times) < args.min_time * 1e3 and len(e2e_times) < MAX_BLOCKS:
        e2e_times.append(e2e_block())
    e2e_ms = float(np.median(e2e_times))
    assert np.isfinite(loss_h.numpy()).all()
    e2e = dict(value=round(world * m * K / (e2e_ms * 1e-3), 1), unit=UNIT,
               h2d_bytes_per_step=int(Xh[0].numel() * Xh[0].element_size() +
                                      yh[0].numel() * yh[0].element_size()),
               d2h_bytes_per_step=int(m * 4), ms_per_step=round(e2e_ms / K, 4),
               blocks=len(e2e_times), timed_s=round(sum(e2e_times) * 1e-3, 3),
               ms_per_step_min=round(min(e2e_times) / K, 4),
               ms_per_step_max=round(max(e2e_times) / K, 4),
               api="%s + olsgd_period_sync, pinned host minibatches (%s rows, int32 labels)"
                   % ("olsgd_local_step_host_bf16" if c["gemm_bf16"] else "olsgd_local_step_host",
                      "bf16" if c["gemm_bf16"] else "fp32"))
    anchor_fusion, summed_floats = anchor_fusion_on, opt.summed_floats
    opt.close()
    del opt, Xd, yd
    torch.cuda.empty_cache()

    # ---- the update and anchor kernels by themselves (the metric's second half)
    if rank == 0 and world == 1 and not args.no_kernel_points:
        roofline["kernels"] += standalone_kernel_rooflines(peaks)

    # ---- with several GPUs: the same job once more with its WORKERS sharded over the ranks
    # (one all-reduce of the anchor sum per period), in the same process group
    sharded = None
    if world > 1 and c["m"] % world == 0 and not local_sgd:
        c_job = dict(c, tau=si.CONFIGS[name]["tau"] if not args.tau else c["tau"])
        s_ms, _, _, _, _ = sharded_job(args, rank, world, c_job, name, K, W)
        sharded = sharded_summary(c_job, P, world, s_ms, K)

    out = None
    if rank == 0:
        cpu = None if args.no_cpu_baseline else cpu_baseline(name, c, X, y, x0, seed)
        resident = X.nbytes + (2 + (1 if c["mu"] else 0) + 1) * m * P * 4
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": round(ms / K, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if c["gemm_bf16"] else "f32", "data": "synthetic",
            "config": {"workload": workload_name(name, c), "m": m, "tau": c["tau"],
                       "batch": B, "dims": c["dims"], "P": P, "gamma": c["gamma"],
                       "alpha": c["alpha"], "beta": c["beta"], "mu": c["mu"],
                       "gemm_mode": c["gemm_bf16"], "method": args.method,
                       "anchor_fusion": bool(anchor_fusion),
                       "worker_sum_formed_by_sync_step_launches_floats": int(summed_floats),
                       "tau_overridden": bool(args.tau),
                       "l2": "no flush: resident inputs+state %.0f MB exceed the %d MB L2"
                             % (resident / 1e6, L2_BYTES >> 20) if resident > L2_BYTES else
                             "state fits in L2 (%.1f MB): steady-state training keeps it there"
                             % (resident / 1e6),
                       "replicas": world},
            "clocks": clocks, "timing": timing, "e2e": e2e, "gpu_launches": int(launches),
            "graph_replays": int(replays),
            "roofline": roofline, "cpu_baseline": cpu,
        }
        if world > 1:
            out["sharded"] = sharded
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out


def run_flat_sweep(args, rank, world):
    """Config 5: fused update and worker-mean kernels on flat parameter vectors with
    external gradients, P x m sweep.  One JSON line; `value` is the largest point."""
    import torch
    from paper_2002_09539_b200 import OverlapLocalSGD
    from paper_2002_09539_b200.build import build

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if rank == 0:
        build()
    c = si.CONFIGS["c5"]
    K, W = args.steps, args.warmup
    peaks = measured_peaks()
    points = []
    Ps = [args.P] if args.P else c["P"]
    ms_ = [args.m] if args.m else c["m"]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
    for P in Ps:
        for m in ms_:
            points.append(flat_point(P, m, K, W, peaks))
    clocks = sampler.stop() if rank == 0 else None
    big = points[-1]
    return {
        "metric": METRIC, "value": big["worker_steps_per_s"], "unit": UNIT, "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": big["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "config 5: update/anchor kernel sweep, flat fp32 parameters, "
                               "external gradients, tau=4, momentum",
                   "value_point": {"P": big["P"], "m": big["m"]},
                   "l2": "no flush; points whose state fits the L2 are flagged in_l2"},
        "clocks": clocks, "e2e": None, "gpu_launches": big["gpu_launches"],
        "roofline": dict(bound="hbm", kernel="update", achieved=big["update_gbs"],
                         peak=peaks["hbm_gbs"], unit="GB/s", frac=big["update_frac_measured"],
                         frac_of_8000=big["update_frac_8000"], traffic=None,
                         peak_source=peaks["source"]),
        "sweep": points,
    }


def sharded_summary(c, P, world, ms, K):
    """The `sharded` record: one m-worker job whose workers are split over `world` GPUs, timed
    over K steps in `ms` milliseconds (max over ranks)."""
    m = c["m"]
    return dict(value=round(m * K / (ms * 1e-3), 1), unit=UNIT, ms_per_step=round(ms / K, 4),
                steps=int(K), scaling="strong", workers_per_gpu=m // world, m=m, n_gpus=int(world),
                allreduce_bytes_per_period=int(P * 4), periods_per_step=round(1.0 / c["tau"], 4),
                collective="ncclAllReduce(sum) of the padded parameter row on the side stream, "
                           "between olsgd_period_sync_begin and olsgd_period_sync_finish")


def sharded_job(args, rank, world, c, name, K, W):
    """ONE m-worker job whose worker dimension is split over the ranks of the (already
    initialised) process group: m / N workers per GPU, the same data set and minibatches as
    the single-GPU job (seed 0, global worker ids).  The only exchange is the sum of Eq. 5, an
    NCCL all-reduce of P floats per period issued on the side stream between
    olsgd_period_sync_begin and olsgd_period_sync_finish, so it overlaps the next period's
    local steps as in the paper.  Returns (ms over K steps as the max over ranks, launches,
    per-class profile, |z| sum, clocks)."""
    import torch
    import torch.distributed as dist
    from paper_2002_09539_b200 import OverlapLocalSGD, class_pairs

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    m = c["m"]
    m_loc, off = m // world, rank * (m // world)
    table = class_pairs(0, m, device="cpu").numpy() if c.get("non_iid") else None
    X, y, x0 = make_inputs(name, 0, table)          # every rank builds the same data set
    Xd = torch.from_numpy(np.ascontiguousarray(X[off:off + m_loc])).cuda()
    yd = torch.from_numpy(np.ascontiguousarray(y[off:off + m_loc])).cuda()
    opt = OverlapLocalSGD(c["kind"], m=m_loc, tau=c["tau"], gamma=c["gamma"], alpha=c["alpha"],
                          beta=c["beta"], mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=Xd, y=yd, worker_offset=off, m_total=m)
    buf = torch.zeros(opt.lib.olsgd_row_floats(opt.ctx), device="cuda")

    def steps(count):
        for _ in range(count):
            opt.local_step()
            if opt.iteration % c["tau"] == 0:
                opt.period_sync_sharded(buf)

    steps(W)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
    dist.barrier()
    torch.cuda.synchronize()
    n0 = opt.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    steps(K)
    opt.main.wait_stream(opt.side)
    e1.record()
    dist.barrier()
    torch.cuda.synchronize()
    ms = max_over_ranks(e0.elapsed_time(e1), world, "cuda")
    launches = opt.launch_count - n0
    clocks = sampler.stop() if rank == 0 else None
    opt.profile_enable(True)
    steps(K)
    prof = opt.profile_read()
    opt.profile_enable(False)
    zsum = float(np.abs(opt.get_params(-1)).sum())
    opt.close()
    del opt, Xd, yd, buf
    torch.cuda.empty_cache()
    return ms, launches, prof, zsum, clocks


def run_sharded(args, rank, world):
    """--shard-workers: the sharded job (see sharded_job) as the whole benchmark.  Total work
    is fixed: strong scaling."""
    import torch
    import torch.distributed as dist
    from paper_2002_09539_b200.build import build

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if not dist.is_initialized():
        if "MASTER_ADDR" not in os.environ:
            os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT="29533")
        dist.init_process_group("nccl", rank=rank, world_size=world,
                                device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build()
    dist.barrier()
    name = args.workload
    c = dict(si.CONFIGS[name])
    if c["gemm_bf16"] and args.gemm_mode:
        c["gemm_bf16"] = args.gemm_mode
    m, K, W = c["m"], args.steps, args.warmup
    if m % world:
        raise SystemExit("--shard-workers needs m (%d) divisible by the number of GPUs (%d)" % (m, world))
    P = n_params(c)
    ms, launches, prof, zsum, clocks = sharded_job(args, rank, world, c, name, K, W)
    out = None
    if rank == 0:
        busy = {k: v for k, v in prof.items() if v[0] > 0}
        out = {
            "metric": METRIC, "value": round(m * K / (ms * 1e-3), 1), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": round(ms / K, 4), "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16" if c["gemm_bf16"] else "f32", "data": "synthetic",
            "config": {"workload": workload_name(name, c), "m": m, "workers_per_gpu": m // world,
                       "tau": c["tau"], "batch": c["batch"], "dims": c["dims"], "P": P,
                       "parallelism": "workers sharded over %d GPU(s), all-reduce of the anchor sum" % world,
                       "allreduce_bytes_per_period": int(P * 4), "anchor_abs_sum": zsum},
            "clocks": clocks, "e2e": None, "gpu_launches": int(launches),
            "sharded": sharded_summary(c, P, world, ms, K),
            "roofline": dict(bound="hbm", kernel=None, traffic=None,
                             class_us_per_step={k: round(v[1] * 1e3 / K, 2) for k, v in busy.items()}),
            "cpu_baseline": None,
        }
    dist.barrier()
    dist.destroy_process_group()
    return out


def max_over_ranks(value, world, device):
    """The slowest rank's value (timings are reported as the max over ranks)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def workload_name(name, c):
    return {"c1": "config 1: linear regression d=64, m=4",
            "c2": "config 2: softmax regression 3072->10, m=16, batch 128",
            "c3": "config 3: MLP 3072-1024-1024-10 bf16, m=16, batch 128, momentum",
            "c4": "config 4: non-IID MLP 3072-512-10 bf16, m=64, batch 64, momentum"}[name]


# ------------------------------------------------------------------ oracle arms (CPU)

def oracle_steps(c, X, y, x0, seed, workers, iters):
    """Run `iters` oracle iterations on the first `workers` workers; returns seconds."""
    from oracle import runner
    t0 = time.perf_counter()
    runner.run_model(c["kind"], c["dims"], X[:workers], y[:workers], x0, m=workers, tau=c["tau"],
                     batch=c["batch"], gamma=c["gamma"], alpha=c["alpha"], beta=c["beta"],
                     mu=c["mu"], seed=seed, iters=iters)
    return time.perf_counter() - t0


def cpu_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count()


def blas_threads(n):
    """Context manager that pins the BLAS thread pool numpy uses to n threads."""
    from threadpoolctl import threadpool_limits
    return threadpool_limits(limits=int(n))


def cpu_baseline(name, c, X, y, x0, seed, budget_s=10.0):
    """The oracle as it stands, timed on a bounded sample of the same workload: with its BLAS
    thread pool set to every core the process may use, and to one core.  The oracle visits the
    workers one after another; the cores are used inside each worker's matrix products."""
    m, cores = c["m"], cpu_cores()
    with blas_threads(cores):
        t1 = oracle_steps(c, X, y, x0, seed, m, 1)              # one full iteration, all workers
        iters = int(max(1, min(c["iters"], budget_s / max(t1, 1e-6))))
        t = oracle_steps(c, X, y, x0, seed, m, iters)
    with blas_threads(1):
        p1 = oracle_steps(c, X, y, x0, seed, 1, 1)              # one worker, one iteration
        w1 = int(max(1, min(m, budget_s / max(p1, 1e-6))))
        it1 = int(max(1, min(c["iters"], budget_s / max(p1 * w1, 1e-6))))
        ts = oracle_steps(c, X, y, x0, seed, w1, it1)
    return dict(value=round(m * iters / t, 2), unit=UNIT, cores=cores, kind="oracle",
                sample="%d iterations of all %d workers (%.1f s), BLAS threads = %d" % (iters, m, t, cores),
                one_core=dict(value=round(w1 * it1 / ts, 2), unit=UNIT, cores=1,
                              sample="%d iterations of %d of the %d workers (%.1f s), BLAS threads = 1"
                                     % (it1, w1, m, ts)))


def run_reference(args, rank, world):
    if rank != 0:
        return None
    name = args.workload
    c = si.CONFIGS[name]
    table = None
    if c.get("non_iid"):
        from oracle import sampling
        table = sampling.class_pairs(0, c["m"])
    X, y, x0 = make_inputs(name, 0, table)
    K, W = args.steps, args.warmup
    m = c["m"]
    # bounded sample: a subset of the workers per step, sized so the run ends in minutes
    with blas_threads(cpu_cores()):
        t1 = oracle_steps(c, X, y, x0, 0, 1, 1)
        budget = 150.0
        workers = int(max(1, min(m, budget / ((K + W) * max(t1, 1e-6)))))
        oracle_steps(c, X, y, x0, 0, workers, W)
        t = oracle_steps(c, X, y, x0, 0, workers, K)
    value = workers * K / t
    sample = "%d of %d workers per step, %d steps" % (workers, m, K)
    return {
        "impl": "reference", "metric": METRIC, "value": round(value, 2), "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": round(t / K * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": workload_name(name, c), "m": m, "tau": c["tau"],
                   "batch": c["batch"], "dims": c["dims"], "sample": sample},
        "cpu_baseline": dict(value=round(value, 2), unit=UNIT, cores=cpu_cores(), kind="oracle",
                             sample=sample),
        "e2e": dict(value=round(value, 2), unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--gemm-mode", type=int, default=0, choices=[0, 1, 2, 3],
                    help="MLP workloads: 1 tensor cores + update fused into the weight-gradient "
                         "GEMM (default), 3 tensor cores + separate update kernel, 2 CUDA cores")
    ap.add_argument("--method", default="overlap", choices=["overlap", "local_sgd", "sync_sgd"],
                    help="overlap: Overlap-Local-SGD (Eq. 3-5, 10-11); local_sgd: blocking periodic "
                         "averaging (Eq. 2); sync_sgd: Eq. 2 with tau = 1")
    ap.add_argument("--shard-workers", action="store_true",
                    help="split the m workers of ONE job over the GPUs (strong scaling) instead of "
                         "running one replica of the job per GPU")
    ap.add_argument("--tau", type=int, default=0,
                    help="c1-c4: override the configuration's period (to measure what a sync costs)")
    ap.add_argument("--P", type=int, default=0, help="c5 only: one parameter count")
    ap.add_argument("--m", type=int, default=0, help="c5 only: one worker count")
    ap.add_argument("--min-time", type=float, default=1.0,
                    help="repeat the timed block of --steps iterations until this many seconds "
                         "have been timed (the median block is reported); 0: one block")
    ap.add_argument("--no-kernel-points", action="store_true",
                    help="skip the stand-alone update/anchor kernel measurements (config 5's "
                         "10M x 16 and 50M x 64 points) that the default line carries")
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip the oracle timing on the host cores (profiling runs)")
    ap.add_argument("--no-anchor-fusion", action="store_true",
                    help="MLP workloads: form the worker sum of Eq. 5 / Eq. 10-11 in the worker-mean "
                         "kernel only (olsgd_set_anchor_fusion(0)), to measure what the fusion buys")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        out = run_reference(args, rank, world)
    elif args.shard_workers:
        out = run_sharded(args, rank, world)
    elif args.workload == "c5":
        out = run_flat_sweep(args, rank, world) if rank == 0 else None
    else:
        out = run_ours(args, rank, world)
    if out is not None:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
