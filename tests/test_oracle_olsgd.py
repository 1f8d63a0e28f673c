"""Pins for oracle.olsgd against what the paper and the mathematics fix:
the matrix form (Eq. 8-9), the algebra of W (Section 2, Appendix A), the
virtual sequence y_k (Appendix A), limiting cases of alpha and beta, and
closed-form linear recursions on noiseless quadratics."""
import numpy as np
import pytest

from oracle import olsgd


def _rand_grads(rng, K, m, d):
    return rng.standard_normal((K, m, d))


# ---------------------------------------------------------------- Eq. 8-9

@pytest.mark.parametrize("m,d,tau,alpha", [(1, 3, 1, 0.5), (3, 5, 2, 0.6), (8, 8, 3, 0.25),
                                           (4, 2, 4, 1.0), (5, 4, 2, 0.0)])
def test_vector_rules_equal_matrix_form_every_iteration(m, d, tau, alpha):
    rng = np.random.default_rng(m * 100 + d)
    gamma, K = 0.07, 13
    x0 = rng.standard_normal(d)
    st = olsgd.OverlapLocalSGD(x0, m, tau, gamma, alpha)
    X = np.tile(x0[:, None], (1, m + 1))                    # Eq. 6
    W = olsgd.mixing_matrix(m, alpha)
    for k, g in enumerate(_rand_grads(rng, K, m, d)):
        G = np.concatenate([g.T, np.zeros((d, 1))], axis=1)  # Eq. 7
        Wk = W if (k + 1) % tau == 0 else np.eye(m + 1)
        X = olsgd.matrix_form_step(X, G, gamma, Wk)
        st.step(g)
        assert np.allclose(st.x.T, X[:, :m], rtol=1e-13, atol=1e-13)
        assert np.allclose(st.z, X[:, m], rtol=1e-13, atol=1e-13)


def test_mixing_matrix_written_out_for_m2():
    # Eq. 9 entry by entry for m = 2, alpha = 0.25
    W = olsgd.mixing_matrix(2, 0.25)
    want = np.array([[0.75, 0.0, 0.375],
                     [0.0, 0.75, 0.375],
                     [0.25, 0.25, 0.25]])
    assert np.array_equal(W, want)


@pytest.mark.parametrize("m,alpha", [(1, 0.5), (4, 0.6), (16, 0.1), (7, 0.9)])
def test_mixing_matrix_algebra(m, alpha):
    W = olsgd.mixing_matrix(m, alpha)
    one = np.ones(m + 1)
    v = np.concatenate([np.full(m, (1 - alpha) / m), [alpha]])
    assert np.allclose(one @ W, one)                 # column-stochastic
    assert np.allclose(W @ v, v)                     # W v = v
    assert v @ one == pytest.approx(1.0)
    # Appendix A: P = (1-alpha) A + alpha b 1^T
    A = np.zeros((m + 1, m + 1))
    A[:m, :m] = np.eye(m)
    A[:m, m] = 1.0 / m
    b = np.zeros(m + 1)
    b[m] = 1.0
    assert np.allclose(W, (1 - alpha) * A + alpha * np.outer(b, one))
    # second-largest eigenvalue modulus of the PageRank-form matrix is <= 1 - alpha,
    # and powers of W converge to v 1^T
    ev = np.sort(np.abs(np.linalg.eigvals(W)))
    assert ev[-1] == pytest.approx(1.0) and ev[-2] <= 1 - alpha + 1e-12
    assert np.allclose(np.linalg.matrix_power(W, 200), np.outer(v, one), atol=1e-9)


# ------------------------------------------------------------ Appendix A

@pytest.mark.parametrize("mu", [0.0, 0.9])
def test_virtual_sequence_descends_by_effective_rate(mu):
    rng = np.random.default_rng(8)
    m, d, tau, gamma, alpha = 5, 6, 3, 0.1, 0.6
    st = olsgd.OverlapLocalSGD(rng.standard_normal(d), m, tau, gamma, alpha, 0.0, mu)
    u = np.zeros((m, d))
    for g in _rand_grads(rng, 17, m, d):
        y = st.virtual_sequence()
        u = mu * u + g
        direction = g + mu * u if mu else g          # the step actually applied
        st.step(g)
        want = y - (1 - alpha) * gamma * direction.mean(axis=0)
        assert np.allclose(st.virtual_sequence(), want, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------- limiting cases

def test_alpha_zero_is_m_independent_sgd_runs():
    rng = np.random.default_rng(9)
    m, d, K, gamma = 4, 5, 11, 0.05
    x0 = rng.standard_normal(d)
    gs = _rand_grads(rng, K, m, d)
    st = olsgd.OverlapLocalSGD(x0, m, 2, gamma, 0.0)
    for g in gs:
        st.step(g)
    for i in range(m):
        x = x0.copy()
        for k in range(K):
            x = x - gamma * gs[k, i]
        assert np.array_equal(st.x[i], x)            # bit for bit


def test_alpha_one_snaps_to_a_frozen_anchor():
    rng = np.random.default_rng(10)
    x0 = rng.standard_normal(4)
    st = olsgd.OverlapLocalSGD(x0, 3, 2, 0.1, 1.0)
    for k, g in enumerate(_rand_grads(rng, 8, 3, 4)):
        st.step(g)
        if (k + 1) % 2 == 0:
            assert np.allclose(st.x, x0) and np.allclose(st.z, x0)


def test_anchor_is_worker_mean_after_every_vanilla_sync_and_frozen_between():
    rng = np.random.default_rng(11)
    st = olsgd.OverlapLocalSGD(rng.standard_normal(6), 7, 3, 0.1, 0.5)
    z_prev = st.z.copy()
    for k, g in enumerate(_rand_grads(rng, 12, 7, 6)):
        st.step(g)
        if (k + 1) % 3 == 0:
            assert np.allclose(st.z, st.x.mean(axis=0), rtol=1e-15, atol=1e-15)
            z_prev = st.z.copy()
        else:
            assert np.array_equal(st.z, z_prev)


def test_pull_back_uses_the_anchor_of_the_previous_period():
    # one-period lag: the pull-back at the end of period a sees z from the end
    # of period a-1, never the fresh mean
    rng = np.random.default_rng(12)
    m, d, tau, gamma, alpha = 3, 4, 2, 0.1, 0.5
    x0 = rng.standard_normal(d)
    gs = _rand_grads(rng, 4, m, d)
    st = olsgd.OverlapLocalSGD(x0, m, tau, gamma, alpha)
    for g in gs[:2]:
        st.step(g)
    half = x0 - gamma * (gs[0] + gs[1])
    assert np.allclose(st.x, (1 - alpha) * half + alpha * x0)      # pulled to z_0 = x0
    z1 = st.x.mean(axis=0)
    x_tau = st.x.copy()
    for g in gs[2:]:
        st.step(g)
    half = x_tau - gamma * (gs[2] + gs[3])
    assert np.allclose(st.x, (1 - alpha) * half + alpha * z1)      # pulled to z_tau


def test_pull_back_contracts_disagreement_by_one_minus_alpha():
    rng = np.random.default_rng(13)
    m, d, gamma, alpha = 6, 5, 0.1, 0.3
    st = olsgd.OverlapLocalSGD(rng.standard_normal(d), m, 1, gamma, alpha)
    for g in _rand_grads(rng, 5, m, d):
        half = st.x - gamma * g
        st.step(g)
        assert np.allclose(st.x - st.x.mean(0), (1 - alpha) * (half - half.mean(0)))


def test_beta_zero_momentum_variant_is_the_vanilla_rule():
    rng = np.random.default_rng(14)
    x0 = rng.standard_normal(5)
    gs = _rand_grads(rng, 12, 4, 5)
    a = olsgd.OverlapLocalSGD(x0, 4, 3, 0.1, 0.6, beta=0.0)
    b = olsgd.OverlapLocalSGD(x0, 4, 3, 0.1, 0.6, beta=1e-300)   # takes the Eq. 10-11 branch
    for g in gs:
        a.step(g)
        b.step(g)
    assert np.allclose(a.z, b.z, rtol=1e-14, atol=1e-15)
    assert np.allclose(a.x, b.x, rtol=1e-14, atol=1e-15)


def test_anchor_momentum_written_out_by_hand():
    # m = 1, d = 1, tau = 1, gamma = 1, alpha = 0.5, beta = 0.5, gradients 1, 1:
    # k=0: x=0-1=-1 -> pull to z=0: -0.5 ; v = 0.5*0 + (-0.5-0) = -0.5 ; z = -0.5
    # k=1: x=-1.5 -> pull to z=-0.5: -1.0 ; v = -0.25 + (-1.0+0.5) = -0.75 ; z = -1.25
    st = olsgd.OverlapLocalSGD(np.zeros(1), 1, 1, 1.0, 0.5, beta=0.5)
    st.step(np.ones((1, 1)))
    assert (st.x[0, 0], st.v[0], st.z[0]) == (-0.5, -0.5, -0.5)
    st.step(np.ones((1, 1)))
    assert (st.x[0, 0], st.v[0], st.z[0]) == (-1.0, -0.75, -1.25)


def test_nesterov_local_step_written_out_by_hand():
    # mu = 0.5, gamma = 1, no sync within these steps; g = 1 then 2
    # u1 = 1, x1 = 0 - (1 + 0.5*1) = -1.5 ; u2 = 0.5 + 2 = 2.5, x2 = -1.5 - (2 + 1.25) = -4.75
    st = olsgd.OverlapLocalSGD(np.zeros(1), 1, 10, 1.0, 0.5, mu=0.5)
    st.step(np.full((1, 1), 1.0))
    assert (st.u[0, 0], st.x[0, 0]) == (1.0, -1.5)
    st.step(np.full((1, 1), 2.0))
    assert (st.u[0, 0], st.x[0, 0]) == (2.5, -4.75)


def test_identical_workers_reduce_to_one_worker():
    rng = np.random.default_rng(15)
    x0 = rng.standard_normal(3)
    gs = rng.standard_normal((9, 1, 3))
    one = olsgd.OverlapLocalSGD(x0, 1, 3, 0.1, 0.6, 0.7, 0.9)
    many = olsgd.OverlapLocalSGD(x0, 5, 3, 0.1, 0.6, 0.7, 0.9)
    for g in gs:
        one.step(g)
        many.step(np.repeat(g, 5, axis=0))
    assert np.allclose(many.x, one.x[0]) and np.allclose(many.z, one.z)


# ---------------------------------------------- closed-form recursions

@pytest.mark.parametrize("tau,alpha", [(1, 0.5), (2, 0.6), (5, 0.3)])
def test_single_worker_noiseless_quadratic_closed_form(tau, alpha):
    # f(x) = h x^2 / 2, c = 1 - gamma h.  With m = 1, z_{a tau} = x_{a tau}, so
    # x_{(a+1) tau} = ((1-alpha) c^tau + alpha) x_{a tau}.
    h, gamma, x0, periods = 2.0, 0.1, 3.0, 6
    c = 1 - gamma * h
    st = olsgd.OverlapLocalSGD(np.array([x0]), 1, tau, gamma, alpha)
    for a in range(1, periods + 1):
        for _ in range(tau):
            st.step(h * st.x)
        want = ((1 - alpha) * c ** tau + alpha) ** a * x0
        assert st.x[0, 0] == pytest.approx(want, rel=1e-13)
        assert st.z[0] == pytest.approx(want, rel=1e-13)


def test_three_periods_by_hand_tau2():
    # h = 1, gamma = 0.5 (c = 0.5), alpha = 0.5, x0 = 16, m = 1, tau = 2:
    # period 1: 16 -> 8 -> 4, pull to z=16: 10, z = 10
    # period 2: 10 -> 5 -> 2.5, pull to z=10: 6.25, z = 6.25
    # period 3: 6.25 -> 3.125 -> 1.5625, pull to 6.25: 3.90625
    st = olsgd.OverlapLocalSGD(np.array([16.0]), 1, 2, 0.5, 0.5)
    seen = []
    for _ in range(6):
        st.step(st.x.copy())
        seen.append(st.x[0, 0])
    assert seen == [8.0, 10.0, 5.0, 6.25, 3.125, 3.90625]
    assert st.z[0] == 3.90625


@pytest.mark.parametrize("beta,mu", [(0.0, 0.0), (0.7, 0.0), (0.0, 0.9), (0.9, 0.9)])
def test_noiseless_quadratics_follow_an_explicit_linear_map(beta, mu):
    # f_i(x) = h (x - c_i)^2 / 2 with full gradients: the whole state
    # (x_1..x_m, u_1..u_m, z, v, 1) evolves by fixed affine maps, one for an
    # ordinary step and one for a sync step.  Build both as matrices here and
    # compare their products with the oracle.
    m, h, gamma, alpha, tau, K = 4, 1.5, 0.08, 0.6, 3, 24
    rng = np.random.default_rng(16)
    cs = rng.standard_normal(m)
    x0 = 2.0
    n = 2 * m + 3
    X, U, Z, V, ONE = slice(0, m), slice(m, 2 * m), 2 * m, 2 * m + 1, 2 * m + 2

    local = np.eye(n)
    for i in range(m):
        xi, ui = i, m + i
        # u' = mu u + h (x - c);  x' = x - gamma (h (x - c) + mu u')
        local[ui, :] = 0
        local[ui, ui], local[ui, xi], local[ui, ONE] = mu, h, -h * cs[i]
        local[xi, :] = 0
        local[xi, xi] = 1 - gamma * h * (1 + mu)
        local[xi, ui] = -gamma * mu * mu
        local[xi, ONE] = gamma * h * (1 + mu) * cs[i]
    pull = np.eye(n)
    for i in range(m):
        pull[i, i], pull[i, Z] = 1 - alpha, alpha
    anchor = np.eye(n)
    # v' = beta v + mean x - z ; z' = z + v'
    anchor[V, :] = 0
    anchor[V, V], anchor[V, Z] = beta, -1.0
    anchor[V, X] = 1.0 / m
    anchor[Z, :] = anchor[V, :]
    anchor[Z, Z] += 1.0
    sync = anchor @ pull @ local

    s = np.zeros(n)
    s[X], s[Z], s[ONE] = x0, x0, 1.0
    st = olsgd.OverlapLocalSGD(np.array([x0]), m, tau, gamma, alpha, beta, mu)
    for k in range(K):
        g = h * (st.x - cs[:, None])
        st.step(g)
        s = (sync if (k + 1) % tau == 0 else local) @ s
        assert np.allclose(st.x[:, 0], s[X], rtol=1e-12, atol=1e-13)
        if mu:
            assert np.allclose(st.u[:, 0], s[U], rtol=1e-12, atol=1e-13)
        assert st.z[0] == pytest.approx(s[Z], rel=1e-12, abs=1e-13)
        if beta:
            assert st.v[0] == pytest.approx(s[V], rel=1e-12, abs=1e-13)


def test_vanilla_mean_recursion_and_fixed_point():
    # per period: xbar' = ((1-alpha) c^tau + alpha) xbar + (1-alpha)(1-c^tau) cbar
    # (after the first sync z = xbar), fixed point cbar
    m, h, gamma, alpha, tau = 5, 1.0, 0.2, 0.5, 2
    rng = np.random.default_rng(17)
    cs = rng.standard_normal(m)
    c = 1 - gamma * h
    st = olsgd.OverlapLocalSGD(np.array([4.0]), m, tau, gamma, alpha)
    xbar = 4.0
    for a in range(200):
        for _ in range(tau):
            st.step(h * (st.x - cs[:, None]))
        xbar = ((1 - alpha) * c ** tau + alpha) * xbar + (1 - alpha) * (1 - c ** tau) * cs.mean()
        assert st.x.mean() == pytest.approx(xbar, rel=1e-11, abs=1e-12)
    assert st.z[0] == pytest.approx(cs.mean(), abs=1e-9)


def test_brute_force_tiny_problem_with_real_minibatches():
    # d = 3 linear regression, m = 2, explicit python loops over samples
    from oracle import runner, sampling
    rng = np.random.default_rng(18)
    m, n, d, B, tau, gamma, alpha, K = 2, 12, 3, 4, 2, 0.1, 0.5, 6
    X = rng.standard_normal((m, n, d))
    y = rng.standard_normal((m, n))
    st, losses, _ = runner.run_model("linreg", [d], X, y, np.zeros(d), m=m, tau=tau, batch=B,
                                     gamma=gamma, alpha=alpha, beta=0.0, mu=0.0, seed=5, iters=K)
    xs = [[0.0] * d for _ in range(m)]
    z = [0.0] * d
    for k in range(K):
        idx = sampling.minibatch_indices(5, m, k, B, n)
        for i in range(m):
            g = [0.0] * d
            for s in idx[i]:
                r = sum(X[i, s, j] * xs[i][j] for j in range(d)) - y[i, s]
                for j in range(d):
                    g[j] += r * X[i, s, j] / B
            xs[i] = [xs[i][j] - gamma * g[j] for j in range(d)]
            if (k + 1) % tau == 0:
                xs[i] = [xs[i][j] - alpha * (xs[i][j] - z[j]) for j in range(d)]
        if (k + 1) % tau == 0:
            z = [sum(xs[i][j] for i in range(m)) / m for j in range(d)]
    assert np.allclose(st.x, np.array(xs), rtol=1e-12, atol=1e-14)
    assert np.allclose(st.z, np.array(z), rtol=1e-12, atol=1e-14)


def test_runner_resumed_from_a_copied_state_continues_the_same_trajectory():
    # the minibatch rule is a function of k alone, so a run split at a period boundary and
    # resumed from copies of (x, u, z, v, k) must give the bits of the unsplit run
    from oracle import runner
    rng = np.random.default_rng(19)
    m, n, d = 3, 20, 4
    X, y = rng.standard_normal((m, n, d)), rng.standard_normal((m, n))
    kw = dict(m=m, tau=2, batch=5, gamma=0.05, alpha=0.6, beta=0.7, mu=0.9, seed=3)
    whole, l_whole, _ = runner.run_model("linreg", [d], X, y, np.zeros(d), iters=10, **kw)
    first, l_a, _ = runner.run_model("linreg", [d], X, y, np.zeros(d), iters=6, **kw)
    again = olsgd.OverlapLocalSGD(np.zeros(d), m, 2, 0.05, 0.6, 0.7, 0.9)
    again.x, again.u, again.z, again.v, again.k = (first.x.copy(), first.u.copy(), first.z.copy(),
                                                   first.v.copy(), first.k)
    second, l_b, _ = runner.run_model("linreg", [d], X, y, None, iters=4, state=again, **kw)
    assert second.k == 10
    assert np.array_equal(second.x, whole.x) and np.array_equal(second.z, whole.z)
    assert np.array_equal(second.v, whole.v) and np.array_equal(second.u, whole.u)
    assert np.array_equal(np.concatenate([l_a, l_b]), l_whole)


# ------------------------------------------------------------ Eq. 2, Local SGD

def test_local_sgd_tau_one_is_sgd_on_the_averaged_gradient():
    # fully synchronous SGD: all workers stay equal and move by the mean gradient
    rng = np.random.default_rng(20)
    x0 = rng.standard_normal(5)
    gs = _rand_grads(rng, 7, 4, 5)
    st = olsgd.LocalSGD(x0, 4, 1, 0.1)
    x = x0.copy()
    for g in gs:
        st.step(g)
        x = x - 0.1 * g.mean(axis=0)
        assert np.allclose(st.x, x, rtol=1e-14, atol=1e-15)


def test_local_sgd_written_out_by_hand():
    # m = 2, tau = 2, gamma = 1, gradients (1, 3) then (2, 0):
    # k=0: x = (-1, -3);  k=1: x = (-3, -3) -> average -3 for both
    st = olsgd.LocalSGD(np.zeros(1), 2, 2, 1.0)
    st.step(np.array([[1.0], [3.0]]))
    assert st.x[:, 0].tolist() == [-1.0, -3.0] and st.z[0] == 0.0
    st.step(np.array([[2.0], [0.0]]))
    assert st.x[:, 0].tolist() == [-3.0, -3.0] and st.z[0] == -3.0


def test_local_sgd_mean_follows_the_mean_gradient_and_workers_agree_after_sync():
    rng = np.random.default_rng(21)
    m, d, tau, gamma = 5, 4, 3, 0.07
    st = olsgd.LocalSGD(rng.standard_normal(d), m, tau, gamma)
    for k, g in enumerate(_rand_grads(rng, 10, m, d)):
        mean_before = st.x.mean(axis=0)
        st.step(g)
        assert np.allclose(st.x.mean(axis=0), mean_before - gamma * g.mean(axis=0), atol=1e-14)
        if (k + 1) % tau == 0:
            assert all(np.array_equal(st.x[i], st.x[0]) for i in range(m))
            assert np.array_equal(st.z, st.x[0])


def test_local_sgd_equals_the_matrix_form_with_full_averaging():
    # Eq. 2 as X_{k+1} = (X_k - gamma G_k) W with W = 1 1^T / m on sync steps
    rng = np.random.default_rng(22)
    m, d, tau, gamma = 4, 3, 2, 0.1
    x0 = rng.standard_normal(d)
    st = olsgd.LocalSGD(x0, m, tau, gamma)
    X = np.tile(x0[:, None], (1, m))
    for k, g in enumerate(_rand_grads(rng, 6, m, d)):
        W = np.full((m, m), 1.0 / m) if (k + 1) % tau == 0 else np.eye(m)
        X = (X - gamma * g.T) @ W
        st.step(g)
        assert np.allclose(st.x.T, X, rtol=1e-13, atol=1e-14)


def test_overlap_with_alpha_one_half_differs_from_local_sgd_only_through_the_lag():
    # one worker: Local SGD is plain SGD; Overlap-Local-SGD with m = 1 pulls toward the
    # previous period's model, so the two differ after the first period
    x0 = np.array([4.0])
    a = olsgd.LocalSGD(x0, 1, 2, 0.25)
    b = olsgd.OverlapLocalSGD(x0, 1, 2, 0.25, 0.5)
    for _ in range(2):
        a.step(a.x.copy())
        b.step(b.x.copy())
    assert a.x[0, 0] == 4.0 * 0.75 ** 2
    assert b.x[0, 0] == 0.5 * 4.0 * 0.75 ** 2 + 0.5 * 4.0
