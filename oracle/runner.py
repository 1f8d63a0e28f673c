"""Glue: run the oracle iteration on a dataset with the sampling rule.

One iteration = for every worker, draw xi_k^(i) (sampling.minibatch_indices),
evaluate g_i at x_k^(i) (models.loss_grad), then olsgd.OverlapLocalSGD.step.

This is test infrastructure (see the package docstring).
"""
import numpy as np

from . import models, olsgd, sampling


def run_model(kind, dims, X, y, x0, *, m, tau, batch, gamma, alpha, beta, mu, seed,
              iters, bf16_operands=False, snapshots=(), local_sgd=False,
              epoch_sampling=False, state=None):
    """Run `iters` iterations; returns (state, losses[iters][m], {k: state copy}).

    X [m][n][d_in], y [m][n]; worker i only ever touches X[i], y[i] (Eq. 1).
    `snapshots` lists iteration counts k at which (x, z, v) are copied out.
    `state`: continue from this state object (its x, u, z, v and k) instead of starting
    from x0; the minibatch rule is a function of k, so a run can be resumed anywhere.
    """
    n = X.shape[1]
    if state is not None:
        st = state
    else:
        st = (olsgd.LocalSGD(x0, m, tau, gamma, mu) if local_sgd
              else olsgd.OverlapLocalSGD(x0, m, tau, gamma, alpha, beta, mu))
    losses = np.zeros((iters, m))
    g = np.zeros_like(st.x)
    snaps = {}
    for t in range(iters):
        k = st.k
        idx = (sampling.minibatch_indices_epoch(seed, m, k, batch, n) if epoch_sampling
               else sampling.minibatch_indices(seed, m, k, batch, n))
        for i in range(m):
            Xb = X[i][idx[i]]
            yb = y[i][idx[i]]
            losses[t, i], g[i] = models.loss_grad(kind, dims, st.x[i], Xb, yb,
                                                  bf16_operands=bf16_operands)
        st.step(g)
        if st.k in snapshots:
            snaps[st.k] = (st.x.copy(), st.z.copy(), st.v.copy())
    return st, losses, snaps


def run_flat(x0, grads, *, m, tau, gamma, alpha, beta, mu, local_sgd=False):
    """External-gradient workload: grads is a sequence of [m][P] arrays."""
    st = (olsgd.LocalSGD(x0, m, tau, gamma, mu) if local_sgd
          else olsgd.OverlapLocalSGD(x0, m, tau, gamma, alpha, beta, mu))
    for g in grads:
        st.step(g)
    return st
