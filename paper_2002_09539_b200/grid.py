"""Sweep of the method's hyper-parameters on a synthetic workload.

    python -m paper_2002_09539_b200.grid [--workload c3] [--iters 400]
           [--taus 1,2,4,8,24] [--alphas 0.5,0.6] [--beta 0.7]

The paper studies how the number of local steps tau and the pull-back rate alpha
trade communication against accuracy (Section 4: tau in {1, 2, 4, 8, 24}, alpha
0.5-0.6, anchor momentum 0.7) and compares with Local SGD.  This script runs the
same grid on one of the synthetic configurations and prints, for every point,
the training loss at the end of the run (mean over the workers and the last 50
iterations), the consensus distance sum_i ||x_i - z||^2 and the throughput.
Everything runs in the library's kernels; nothing here touches the CPU oracle.
"""
import argparse
import time

import numpy as np
import torch

import synth_inputs as si
from . import OverlapLocalSGD, class_pairs


def run_point(c, X, y, x0, *, tau, alpha, beta, local_sgd, iters):
    opt = OverlapLocalSGD(c["kind"], m=c["m"], tau=tau, gamma=c["gamma"], alpha=alpha, beta=beta,
                          mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=X, y=y, local_sgd=local_sgd)
    loss = torch.zeros((iters, c["m"]), device="cuda")
    opt.run(min(10, iters))                     # warm-up of the kernels, then a fresh context
    opt.close()
    opt = OverlapLocalSGD(c["kind"], m=c["m"], tau=tau, gamma=c["gamma"], alpha=alpha, beta=beta,
                          mu=c["mu"], batch=c["batch"], seed=0, dims=c["dims"],
                          gemm_bf16=c["gemm_bf16"], x0=x0, X=X, y=y, local_sgd=local_sgd)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    opt.run(iters, loss)
    opt.join()
    dt = time.perf_counter() - t0
    tail = float(loss[-50:].mean())
    first = float(loss[0].mean())
    dist = opt.consensus_distance()
    opt.close()
    return dict(first=first, tail=tail, consensus=dist, wsps=c["m"] * iters / dt)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4"])
    ap.add_argument("--iters", type=int, default=400)
    ap.add_argument("--taus", default="1,2,4,8,24")
    ap.add_argument("--alphas", default="0.5,0.6")
    ap.add_argument("--beta", type=float, default=0.7)
    args = ap.parse_args()
    c = dict(si.CONFIGS[args.workload])
    table = class_pairs(0, c["m"], device="cpu").numpy() if c.get("non_iid") else None
    Xh, yh = si.mixture_data(0, c["m"], c["n"], c["dims"][0], table)
    x0 = si.model_init(0, c["kind"], c["dims"])
    X, y = torch.from_numpy(Xh).cuda(), torch.from_numpy(yh).cuda()
    taus = [int(t) for t in args.taus.split(",")]
    alphas = [float(a) for a in args.alphas.split(",")]
    print("workload %s, %d iterations, m = %d, gamma = %g, local momentum %g, anchor momentum %g"
          % (args.workload, args.iters, c["m"], c["gamma"], c["mu"], args.beta))
    print("| method | tau | alpha | loss (first) | loss (last 50) | consensus distance | worker-steps/s |")
    print("|---|---|---|---|---|---|---|")
    for tau in taus:
        iters = (args.iters // tau) * tau
        r = run_point(c, X, y, x0, tau=tau, alpha=0.0, beta=0.0, local_sgd=True, iters=iters)
        name = "sync SGD (Eq. 2, tau = 1)" if tau == 1 else "Local SGD (Eq. 2)"
        print("| %s | %d | - | %.4f | %.4f | %.3e | %.0f |" % (name, tau, r["first"], r["tail"],
                                                          r["consensus"], r["wsps"]))
        for alpha in alphas:
            r = run_point(c, X, y, x0, tau=tau, alpha=alpha, beta=args.beta, local_sgd=False,
                          iters=iters)
            print("| Overlap-Local-SGD | %d | %.2f | %.4f | %.4f | %.3e | %.0f |"
                  % (tau, alpha, r["first"], r["tail"], r["consensus"], r["wsps"]))


if __name__ == "__main__":
    main()
