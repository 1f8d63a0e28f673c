"""Writes the stored expected values of the full-length MLP configurations.

Calls only the CPU oracle and the seeded input generators.  Usage:
    python tests/golden/make_golden.py c3 [c4 ...]
    python tests/golden/make_golden.py c3 --perturb     (writes c3_perturbed.json)
With --perturb the run starts from x0 with 1e-7 added to its first entry: the
difference to the unperturbed result measures how far two correct fp64 runs of
the same configuration drift apart, i.e. what no parity tolerance can beat.
Each run takes tens of minutes (fp64, full data set, every iteration) and
writes tests/golden/<name>_final.json with the final objective F of Eq. 1
evaluated on every worker's whole partition at the mean model and at the
anchor, the trailing minibatch losses, and a few summary numbers of the state.
"""
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import synth_inputs as si                      # noqa: E402
from oracle import models, runner, sampling    # noqa: E402

SEED = 0


def main(names):
    perturb = "--perturb" in names
    names = [n for n in names if not n.startswith("--")]
    for name in names:
        c = si.CONFIGS[name]
        table = sampling.class_pairs(SEED, c["m"]) if c["non_iid"] else None
        X, y = si.mixture_data(SEED, c["m"], c["n"], c["dims"][0], table)
        x0 = si.model_init(SEED, c["kind"], c["dims"])
        if perturb:
            x0[0] += 1e-7
        t0 = time.time()
        st, losses, _ = runner.run_model(
            c["kind"], c["dims"], X, y, x0, m=c["m"], tau=c["tau"], batch=c["batch"],
            gamma=c["gamma"], alpha=c["alpha"], beta=c["beta"], mu=c["mu"], seed=SEED,
            iters=c["iters"])
        xbar = st.mean_model()
        probe = np.linspace(0, xbar.size - 1, 16).astype(np.int64)
        out = {
            "config": name, "seed": SEED, "iters": c["iters"], "x0_perturbation": 1e-7 if perturb else 0.0,
            "oracle_seconds": round(time.time() - t0, 1),
            "F_mean_model": models.full_objective(c["kind"], c["dims"], xbar, X, y),
            "F_anchor": models.full_objective(c["kind"], c["dims"], st.z, X, y),
            "minibatch_loss_mean_every_50": [float(v) for v in losses.mean(axis=1)[49::50]],
            # mean over workers AND over each block of 50 iterations: a far less noisy
            # statistic of the trajectory than one iteration's loss
            "minibatch_loss_block_mean_50": [float(losses[b:b + 50].mean())
                                             for b in range(0, losses.shape[0] - 49, 50)],
            "minibatch_loss_last10_mean": float(losses[-10:].mean()),
            "norm2_mean_model": float(np.linalg.norm(xbar)),
            "norm2_anchor": float(np.linalg.norm(st.z)),
            "consensus_sq": float(((st.x - st.z) ** 2).sum()),
            "probe_index": [int(p) for p in probe],
            "probe_mean_model": [float(v) for v in xbar[probe]],
            "probe_anchor": [float(v) for v in st.z[probe]],
        }
        with open(os.path.join(HERE, name + ("_perturbed.json" if perturb else "_final.json")), "w") as f:
            json.dump(out, f, indent=1)
            f.write("\n")
        print(name, "done in", out["oracle_seconds"], "s", flush=True)


if __name__ == "__main__":
    main(sys.argv[1:] or ["c3", "c4"])
