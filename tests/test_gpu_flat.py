"""Fused update (Eq. 3-4) and worker-mean anchor (Eq. 5, 10-11) kernels against
the oracle on external gradients: element by element, sizes that span several
tiles with a ragged tail, all four momentum combinations."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import synth_inputs as si
from oracle import runner
from helpers import max_rel_err, state_err, to_dev

TOL = 1e-5   # max relative parameter error of the fp32 path


def _run_pair(P, m, tau, gamma, alpha, beta, mu, iters, seed=0, overlap=True, std=0.1):
    from paper_2002_09539_b200 import OverlapLocalSGD
    x0 = si.flat_init(seed, P)
    grads = [si.flat_grads(seed, k, m, P, std) for k in range(iters)]
    st = runner.run_flat(x0, grads, m=m, tau=tau, gamma=gamma, alpha=alpha, beta=beta, mu=mu)
    opt = OverlapLocalSGD("flat", m=m, tau=tau, gamma=gamma, alpha=alpha, beta=beta, mu=mu,
                          flat_P=P, x0=x0, overlap=overlap)
    for k in range(iters):
        opt.local_step_with_grads(to_dev(grads[k]))
        if (k + 1) % tau == 0:
            opt.period_sync()
    return opt, st


@pytest.mark.parametrize("beta,mu", [(0.0, 0.0), (0.9, 0.0), (0.0, 0.9), (0.9, 0.9)])
@pytest.mark.parametrize("P,m,tau", [(4 * 256 * 3 + 7, 8, 4), (1, 1, 1), (5, 3, 2), (1000003, 16, 4),
                                     (70001, 37, 3), (4096, 64, 1)])
def test_flat_parity(P, m, tau, beta, mu):
    opt, st = _run_pair(P, m, tau, 0.05, 0.5, beta, mu, iters=3 * tau + 1)
    assert state_err(opt, st) <= TOL
    v = opt.get_params(-2)
    if beta:
        # v is a difference of nearly equal vectors: its error is measured on the scale of z
        assert np.abs(v - st.v).max() <= TOL * max(np.abs(st.z).max(), np.abs(st.v).max())
    if mu:
        u0 = opt.get_params(-5)
        assert max_rel_err([u0], [st.u[0]]) <= TOL
        ul = opt.get_params(-5 - (m - 1))
        assert max_rel_err([ul], [st.u[m - 1]]) <= TOL
    y = opt.get_params(-3)
    assert max_rel_err([y], [st.virtual_sequence()]) <= TOL
    xbar = opt.get_params(-4)
    assert max_rel_err([xbar], [st.mean_model()]) <= TOL


def _run_bits(P, m, tau, beta, mu, iters, fusion, grads, x0):
    from paper_2002_09539_b200 import OverlapLocalSGD
    opt = OverlapLocalSGD("flat", m=m, tau=tau, gamma=0.05, alpha=0.5, beta=beta, mu=mu, flat_P=P, x0=x0)
    opt.set_anchor_fusion(fusion)
    for k in range(iters):
        opt.local_step_with_grads(grads[k])
        if (k + 1) % tau == 0:
            opt.period_sync()
    return opt


# rows long enough that the sync step's update launch forms the worker sums itself (one
# thread per 16 bytes and slice must give every multiprocessor work): S = 1, 2, 2 and 4
# slices, ragged tails and ragged slices
@pytest.mark.parametrize("beta,mu", [(0.0, 0.0), (0.9, 0.9)])
@pytest.mark.parametrize("P,m,tau", [(2_500_003, 5, 2), (1_300_003, 16, 4), (300_001, 37, 1),
                                     (700_002, 64, 2)])
def test_update_kernel_forms_the_worker_sum_on_long_rows(P, m, tau, beta, mu):
    iters = 2 * tau + 1
    x0 = si.flat_init(3, P)
    host = [si.flat_grads(3, k, m, P, 0.1) for k in range(iters)]
    grads = [to_dev(g) for g in host]
    on = _run_bits(P, m, tau, beta, mu, iters, True, grads, x0)
    off = _run_bits(P, m, tau, beta, mu, iters, False, grads, x0)
    assert on.anchor_fusion and not off.anchor_fusion
    assert on.summed_floats == P and off.summed_floats == 0
    for a, b in zip(on.state(), off.state()):
        assert np.array_equal(a, b)                      # same summation order, same bits
    st = runner.run_flat(x0, host, m=m, tau=tau, gamma=0.05, alpha=0.5, beta=beta, mu=mu)
    assert state_err(on, st) <= TOL


@pytest.mark.parametrize("P,m", [(50021, 16), (2_000_001, 3)])
def test_short_rows_and_few_workers_leave_the_worker_sum_to_the_anchor_kernel(P, m):
    tau = 2
    x0 = si.flat_init(4, P)
    grads = [to_dev(si.flat_grads(4, k, m, P, 0.1)) for k in range(tau)]
    opt = _run_bits(P, m, tau, 0.9, 0.9, tau, True, grads, x0)
    assert opt.anchor_fusion and opt.summed_floats == 0


def test_hundred_iterations_stay_within_tolerance():
    opt, st = _run_pair(50021, 16, 4, 0.05, 0.5, 0.9, 0.9, iters=100)
    assert state_err(opt, st) <= TOL


def test_anchor_is_exact_mean_and_frozen_between_syncs():
    from paper_2002_09539_b200 import OverlapLocalSGD
    P, m, tau = 3000, 8, 3
    x0 = si.flat_init(1, P)
    opt = OverlapLocalSGD("flat", m=m, tau=tau, gamma=0.1, alpha=0.6, flat_P=P, x0=x0)
    z_prev = opt.get_params(-1).copy()
    assert np.array_equal(z_prev, x0)
    for k in range(2 * tau):
        opt.local_step_with_grads(to_dev(si.flat_grads(1, k, m, P)))
        if (k + 1) % tau == 0:
            opt.period_sync()
            x, z, _ = opt.state()
            assert np.abs(z - x.astype(np.float64).mean(0)).max() <= 2e-7 * np.abs(z).max()
            z_prev = z
        else:
            assert np.array_equal(opt.get_params(-1), z_prev)


def test_alpha_zero_and_alpha_one():
    from paper_2002_09539_b200 import OverlapLocalSGD
    P, m, tau = 2049, 4, 2
    x0 = si.flat_init(2, P)
    grads = [si.flat_grads(2, k, m, P) for k in range(4)]
    a0 = OverlapLocalSGD("flat", m=m, tau=tau, gamma=0.1, alpha=0.0, flat_P=P, x0=x0)
    a1 = OverlapLocalSGD("flat", m=m, tau=tau, gamma=0.1, alpha=1.0, flat_P=P, x0=x0)
    for k, g in enumerate(grads):
        for o in (a0, a1):
            o.local_step_with_grads(to_dev(g))
            if (k + 1) % tau == 0:
                o.period_sync()
    x, _, _ = a0.state()
    want = x0[None, :].astype(np.float64) - 0.1 * np.sum(grads, axis=0, dtype=np.float64)
    assert max_rel_err(list(x), list(want)) <= TOL       # m independent SGD runs
    x, z, _ = a1.state()
    # x - 1.0 * (x - z) returns z up to one rounding of the difference
    assert max_rel_err([z] + list(x), [x0] * (m + 1)) <= 1e-6


def test_overlapped_and_serial_streams_give_identical_bits():
    a, _ = _run_pair(123457, 8, 2, 0.05, 0.5, 0.9, 0.9, iters=9, overlap=True)
    b, _ = _run_pair(123457, 8, 2, 0.05, 0.5, 0.9, 0.9, iters=9, overlap=False)
    xa, za, va = a.state()
    xb, zb, vb = b.state()
    assert np.array_equal(xa, xb) and np.array_equal(za, zb) and np.array_equal(va, vb)


def test_call_order_is_enforced():
    from paper_2002_09539_b200 import OverlapLocalSGD, OlsgdError
    P, m = 64, 2
    opt = OverlapLocalSGD("flat", m=m, tau=2, gamma=0.1, alpha=0.5, flat_P=P, x0=np.zeros(P, np.float32))
    g = torch.zeros((m, P), device="cuda")
    with pytest.raises(OlsgdError) as e:
        opt.period_sync()                       # no period has ended
    assert e.value.status == 2
    opt.local_step_with_grads(g)
    with pytest.raises(OlsgdError):
        opt.period_sync()                       # mid-period
    opt.local_step_with_grads(g)
    with pytest.raises(OlsgdError):
        opt.local_step_with_grads(g)            # sync is due
    opt.period_sync()
    with pytest.raises(OlsgdError):
        opt.period_sync()                       # only once per period
    with pytest.raises(OlsgdError):
        opt.local_step()                        # wrong entry point for FLAT
    with pytest.raises(OlsgdError):
        opt.get_params(m)
    assert opt.iteration == 2
    opt.local_step_with_grads(g)
    assert opt.iteration == 3 and opt.launch_count >= 4


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # no fault, no hang: one thread waits 20 ms on a barrier nothing arrives on, gives up,
    # and the host reads OLSGD_ETIMEOUT at the next join
    import time
    from paper_2002_09539_b200 import OverlapLocalSGD, OlsgdError
    P, m = 1024, 2
    x0 = si.flat_init(3, P)
    opt = OverlapLocalSGD("flat", m=m, tau=2, gamma=0.1, alpha=0.5, flat_P=P, x0=x0)
    g = to_dev(si.flat_grads(3, 0, m, P))
    opt.local_step_with_grads(g)
    opt.join()
    t0 = time.time()
    opt.selftest_wait_timeout(20)
    with pytest.raises(OlsgdError) as e:
        opt.join()
    assert e.value.status == 5                      # OLSGD_ETIMEOUT
    assert time.time() - t0 < 5.0
    with pytest.raises(OlsgdError):
        opt.get_params(0)                           # still reported until cleared
    opt.clear_status()
    opt.join()
    opt.local_step_with_grads(g)                    # the context works as before
    opt.period_sync()
    x = opt.get_params(0)
    want = x0.astype(np.float64) - 0.1 * 2 * g[0].cpu().numpy().astype(np.float64)
    want = want - 0.5 * (want - x0)
    assert max_rel_err([x], [want]) <= 1e-6


@pytest.mark.parametrize("P,m,tau,mu", [(4 * 256 * 3 + 7, 8, 4, 0.0), (70001, 37, 3, 0.9),
                                        (1000003, 16, 1, 0.9), (5, 3, 2, 0.0)])
def test_local_sgd_mode_parity(P, m, tau, mu):
    # Eq. 2: blocking periodic averaging; tau = 1 is fully synchronous SGD
    from paper_2002_09539_b200 import OverlapLocalSGD, OlsgdError
    iters = 3 * tau + 1
    x0 = si.flat_init(4, P)
    grads = [si.flat_grads(4, k, m, P) for k in range(iters)]
    st = runner.run_flat(x0, grads, m=m, tau=tau, gamma=0.05, alpha=0.5, beta=0.0, mu=mu,
                         local_sgd=True)
    opt = OverlapLocalSGD("flat", m=m, tau=tau, gamma=0.05, alpha=0.5, mu=mu, flat_P=P, x0=x0,
                          local_sgd=True)
    for k in range(iters):
        opt.local_step_with_grads(to_dev(grads[k]))
        if (k + 1) % tau == 0:
            x, z, _ = opt.state()
            assert all(np.array_equal(x[i], x[0]) for i in range(m))    # all workers agree
            assert np.array_equal(z, x[0])
            with pytest.raises(OlsgdError):
                opt.period_sync()                                        # never due in this mode
    assert state_err(opt, st) <= TOL
