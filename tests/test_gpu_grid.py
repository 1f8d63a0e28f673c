"""The hyper-parameter grid module (the synthetic stand-in for the paper's Section 4 figures):
it writes its curves, and what it writes is the method's trajectory."""
import csv
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import synth_inputs as si
from oracle import runner
from helpers import to_dev


def _rows(path):
    with open(path) as f:
        return list(csv.DictReader(line for line in f if not line.startswith("#")))


def test_grid_writes_loss_and_consensus_curves_that_follow_the_oracle(tmp_path):
    from paper_2002_09539_b200 import grid
    dims, m, n, batch, iters, tau, alpha, beta = [128, 128, 10], 4, 96, 64, 40, 2, 0.6, 0.7
    c = dict(kind="mlp", dims=dims, m=m, n=n, batch=batch, tau=tau, gamma=0.05, alpha=alpha,
             beta=beta, mu=0.9, gemm_bf16=1)
    X, y = si.mixture_data(31, m, n, dims[0])
    x0 = si.model_init(31, "mlp", dims)
    points = [("Overlap-Local-SGD", tau, alpha, beta, False), ("Local SGD (Eq. 2)", tau, 0.0, 0.0, True)]
    res = grid.run_grid(c, to_dev(X), to_dev(y), x0, points, iters, str(tmp_path), "tiny",
                        consensus_stride=1)
    assert set(res) == {("Overlap-Local-SGD", tau, alpha), ("Local SGD (Eq. 2)", tau, 0.0)}
    loss_rows = _rows(os.path.join(tmp_path, "hyperparameter_grid_tiny_loss.csv"))
    cons_rows = _rows(os.path.join(tmp_path, "hyperparameter_grid_tiny_consensus.csv"))
    assert os.path.exists(os.path.join(tmp_path, "hyperparameter_grid_tiny.md"))
    assert len(loss_rows) == 2 * (iters // grid.LOSS_BLOCK) and len(cons_rows) == 2 * (iters // tau)

    # the Overlap-Local-SGD point against the oracle (same operand rounding), minibatches of
    # the index rule with seed 0 as the module uses
    st_curve, snaps = [], {}
    st, lo, snaps = runner.run_model("mlp", dims, X, y, x0, m=m, tau=tau, batch=batch, gamma=0.05,
                                     alpha=alpha, beta=beta, mu=0.9, seed=0, iters=iters,
                                     bf16_operands=True, snapshots=range(tau, iters + 1, tau))
    want_loss = lo.mean(axis=1).reshape(-1, grid.LOSS_BLOCK).mean(axis=1)
    got_loss = np.array([float(r["loss"]) for r in loss_rows if r["method"] == "Overlap-Local-SGD"])
    assert np.abs(got_loss - want_loss).max() <= 2e-2 * np.abs(want_loss).max()
    got_cons = {int(r["iteration"]): float(r["consensus_distance"]) for r in cons_rows
                if r["method"] == "Overlap-Local-SGD"}
    for k, (xs, z, _) in snaps.items():
        want = float(((xs - z[None, :]) ** 2).sum())
        assert abs(got_cons[k] - want) <= 5e-2 * want, (k, got_cons[k], want)
    # Local SGD: all workers equal the average right after every averaging step
    assert all(float(r["consensus_distance"]) == 0.0 for r in cons_rows if r["method"] != "Overlap-Local-SGD")
    assert got_loss[-1] < got_loss[0]
