"""Sweep of the method's hyper-parameters on a synthetic workload, as curves.

    python -m paper_2002_09539_b200.grid [--workload c3] [--iters 300]
           [--taus 1,2,4,8,24] [--alphas 0.5,0.6] [--beta 0.7] [--out profiles]

The paper studies how the number of local steps tau and the pull-back rate alpha
trade communication against accuracy (Section 4, Fig. 4-5 and Tables 1-2: tau in
{1, 2, 4, 8, 24}, alpha 0.5-0.6, anchor momentum 0.7) and compares with Local SGD
and fully synchronous SGD.  This module runs the same grid on one of the synthetic
configurations and writes, for every (method, tau, alpha):

  <out>/hyperparameter_grid_<workload>_loss.csv        training loss against iterations: the
        minibatch loss averaged over the workers and over blocks of ten iterations
  <out>/hyperparameter_grid_<workload>_consensus.csv   the consensus distance
        sum_i ||x_i - z||^2 right after every anchor refresh (every averaging step for
        Local SGD, where it is zero by construction)
  <out>/hyperparameter_grid_<workload>.md              the end-of-run table

It is the synthetic stand-in for the paper's figures, not a reproduction of their numbers
(no CIFAR-10, no ResNet-18).  Everything runs in the library's kernels; nothing here
touches the CPU oracle.
"""
import argparse
import os
import time

import numpy as np
import torch

import synth_inputs as si
from . import OverlapLocalSGD, class_pairs

LOSS_BLOCK = 10


def run_point(c, X, y, x0, *, tau, alpha, beta, local_sgd, iters):
    """One grid point.  Returns the per-iteration worker-mean loss [iters], the consensus
    distance after every sync [(iteration, value)], and the wall-clock throughput."""
    opt = OverlapLocalSGD(c["kind"], m=c["m"], tau=tau, gamma=c["gamma"], alpha=alpha, beta=beta,
                          mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=X, y=y, local_sgd=local_sgd)
    loss = torch.zeros((iters, c["m"]), device="cuda")
    consensus = []
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    k = 0
    while k < iters:
        step = min(tau, iters - k)
        opt.run(step, loss[k:k + step])
        k += step
        if k % tau == 0:
            consensus.append((k, opt.consensus_distance()))     # joins the streams
    opt.join()
    dt = time.perf_counter() - t0
    opt.close()
    return loss.mean(dim=1).cpu().numpy().astype(np.float64), consensus, c["m"] * iters / dt


def grid_points(taus, alphas, beta):
    """(label, tau, alpha, beta, local_sgd) in the order of the paper's tables."""
    pts = []
    for tau in taus:
        pts.append(("sync SGD (Eq. 2, tau = 1)" if tau == 1 else "Local SGD (Eq. 2)", tau, 0.0, 0.0, True))
        for alpha in alphas:
            pts.append(("Overlap-Local-SGD", tau, alpha, beta, False))
    return pts


def run_grid(c, X, y, x0, points, iters, out_dir=None, tag="grid", command="", consensus_stride=10):
    """Runs the points, returns {(label, tau, alpha): dict(loss, consensus, wsps)} and, with
    out_dir, writes the two CSV files and the table.  The consensus file keeps every
    max(1, consensus_stride // tau)-th anchor refresh of a point (all of them are returned)."""
    results = {}
    for label, tau, alpha, beta, local in points:
        n = (iters // tau) * tau
        loss, cons, wsps = run_point(c, X, y, x0, tau=tau, alpha=alpha, beta=beta, local_sgd=local,
                                     iters=n)
        results[(label, tau, alpha)] = dict(loss=loss, consensus=cons, wsps=wsps, beta=beta, iters=n)
    if out_dir is not None:
        os.makedirs(out_dir, exist_ok=True)
        head = ("# written by python -m paper_2002_09539_b200.grid%s\n"
                "# m = %d workers, batch %d, gamma = %g, local momentum %g; synthetic data\n"
                % ((" " + command) if command else "", c["m"], c["batch"], c["gamma"], c["mu"]))
        with open(os.path.join(out_dir, "hyperparameter_grid_%s_loss.csv" % tag), "w") as f:
            f.write(head)
            f.write("# loss: minibatch loss, mean over the workers and over iterations "
                    "[iteration - %d, iteration)\n" % LOSS_BLOCK)
            f.write("method,tau,alpha,beta,iteration,loss\n")
            for (label, tau, alpha), r in results.items():
                for b in range(len(r["loss"]) // LOSS_BLOCK):
                    f.write("%s,%d,%g,%g,%d,%.6f\n" % (label, tau, alpha, r["beta"], (b + 1) * LOSS_BLOCK,
                                                       r["loss"][b * LOSS_BLOCK:(b + 1) * LOSS_BLOCK].mean()))
        with open(os.path.join(out_dir, "hyperparameter_grid_%s_consensus.csv" % tag), "w") as f:
            f.write(head)
            f.write("# consensus_distance: sum_i ||x_i - z||^2 after the anchor refresh that closes "
                    "iteration `iteration` (every max(1, %d // tau)-th refresh is listed)\n" % consensus_stride)
            f.write("method,tau,alpha,beta,iteration,consensus_distance\n")
            for (label, tau, alpha), r in results.items():
                keep = max(1, consensus_stride // tau)
                for k, v in r["consensus"]:
                    if (k // tau) % keep == 0:
                        f.write("%s,%d,%g,%g,%d,%.6e\n" % (label, tau, alpha, r["beta"], k, v))
        with open(os.path.join(out_dir, "hyperparameter_grid_%s.md" % tag), "w") as f:
            f.write(head.replace("# ", "").replace("\n", "  \n"))
            f.write("\nLoss = training minibatch loss, mean over the workers; throughput by wall clock, "
                    "including one consensus-distance reduction per period.\n\n")
            f.write("| method | tau | alpha | loss (first) | loss (last 50) | consensus distance (end) "
                    "| worker-steps/s |\n|---|---|---|---|---|---|---|\n")
            for (label, tau, alpha), r in results.items():
                f.write("| %s | %d | %s | %.4f | %.4f | %.3e | %.0f |\n"
                        % (label, tau, "-" if label != "Overlap-Local-SGD" else "%.2f" % alpha,
                           r["loss"][0], r["loss"][-50:].mean(),
                           r["consensus"][-1][1] if r["consensus"] else float("nan"), r["wsps"]))
    return results


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4"])
    ap.add_argument("--iters", type=int, default=300)
    ap.add_argument("--taus", default="1,2,4,8,24")
    ap.add_argument("--alphas", default="0.5,0.6")
    ap.add_argument("--beta", type=float, default=0.7)
    ap.add_argument("--out", default="profiles")
    ap.add_argument("--consensus-stride", type=int, default=10,
                    help="list the consensus distance about every this many iterations")
    args = ap.parse_args()
    c = dict(si.CONFIGS[args.workload])
    table = class_pairs(0, c["m"], device="cpu").numpy() if c.get("non_iid") else None
    Xh, yh = si.mixture_data(0, c["m"], c["n"], c["dims"][0], table)
    x0 = si.model_init(0, c["kind"], c["dims"])
    X, y = torch.from_numpy(Xh).cuda(), torch.from_numpy(yh).cuda()
    taus = [int(t) for t in args.taus.split(",")]
    alphas = [float(a) for a in args.alphas.split(",")]
    command = "--workload %s --iters %d --taus %s --alphas %s --beta %g" % (
        args.workload, args.iters, args.taus, args.alphas, args.beta)
    res = run_grid(c, X, y, x0, grid_points(taus, alphas, args.beta), args.iters, args.out,
                   args.workload, command, args.consensus_stride)
    for (label, tau, alpha), r in res.items():
        print("%-28s tau %2d alpha %.2f  loss %.4f -> %.4f  consensus %.3e  %.0f worker-steps/s"
              % (label, tau, alpha, r["loss"][0], r["loss"][-50:].mean(),
                 r["consensus"][-1][1] if r["consensus"] else float("nan"), r["wsps"]))


if __name__ == "__main__":
    main()
