"""The worker dimension sharded over two contexts (as it would be over two GPUs), emulated
on one GPU in one process: each context holds half of the workers, the only exchange is the
sum of Eq. 5, formed here by adding the two partial-sum buffers where a multi-GPU run calls
all-reduce.  No kernel waits on another; the host orders the stages."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import synth_inputs as si
from oracle import runner, sampling
from helpers import max_rel_err, to_dev


def _sync_two(a, b, bufa, bufb):
    a.period_sync_begin(bufa)
    b.period_sync_begin(bufb)
    torch.cuda.synchronize()
    total = bufa + bufb                    # stands in for the all-reduce
    torch.cuda.synchronize()
    a.period_sync_finish(total)
    b.period_sync_finish(total)
    return total


@pytest.mark.parametrize("beta,mu", [(0.0, 0.0), (0.9, 0.9)])
def test_two_shards_of_flat_workers_equal_the_oracle(beta, mu):
    from paper_2002_09539_b200 import OverlapLocalSGD, OlsgdError
    P, m, tau, iters = 70001, 6, 2, 7
    x0 = si.flat_init(5, P)
    grads = [si.flat_grads(5, k, m, P) for k in range(iters)]
    st = runner.run_flat(x0, grads, m=m, tau=tau, gamma=0.05, alpha=0.6, beta=beta, mu=mu)
    kw = dict(tau=tau, gamma=0.05, alpha=0.6, beta=beta, mu=mu, flat_P=P, x0=x0, m_total=m)
    a = OverlapLocalSGD("flat", m=4, worker_offset=0, **kw)
    b = OverlapLocalSGD("flat", m=2, worker_offset=4, **kw)
    n = a.lib.olsgd_row_floats(a.ctx)
    bufa, bufb = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    for k in range(iters):
        a.local_step_with_grads(to_dev(grads[k][:4]))
        b.local_step_with_grads(to_dev(grads[k][4:]))
        if (k + 1) % tau == 0:
            with pytest.raises(OlsgdError):
                a.period_sync()            # a shard cannot refresh the anchor on its own
            _sync_two(a, b, bufa, bufb)
    xa, za, va = a.state()
    xb, zb, vb = b.state()
    assert np.array_equal(za, zb) and np.array_equal(va, vb)     # both shards hold the same anchor
    got = [xa[i] for i in range(4)] + [xb[i] for i in range(2)] + [za]
    want = [st.x[i] for i in range(m)] + [st.z]
    assert max_rel_err(got, want) <= 1e-5


@pytest.mark.parametrize("beta,mu", [(0.0, 0.0), (0.9, 0.9)])
def test_shards_whose_update_launch_forms_the_partial_sums(beta, mu):
    """Rows long enough that each shard's sync-step update kernel adds up its own workers:
    olsgd_period_sync_begin then only combines the slices.  Same bits as with the sum left to
    the worker-mean kernel, and the oracle's m-worker trajectory."""
    from paper_2002_09539_b200 import OverlapLocalSGD
    P, m, tau, iters = 1_300_003, 24, 2, 5
    x0 = si.flat_init(7, P)
    host = [si.flat_grads(7, k, m, P) for k in range(iters)]
    st = runner.run_flat(x0, host, m=m, tau=tau, gamma=0.05, alpha=0.6, beta=beta, mu=mu)
    kw = dict(tau=tau, gamma=0.05, alpha=0.6, beta=beta, mu=mu, flat_P=P, x0=x0, m_total=m)
    states = {}
    for fusion in (True, False):
        a = OverlapLocalSGD("flat", m=16, worker_offset=0, **kw)
        b = OverlapLocalSGD("flat", m=8, worker_offset=16, **kw)
        a.set_anchor_fusion(fusion)
        b.set_anchor_fusion(fusion)
        n = a.lib.olsgd_row_floats(a.ctx)
        bufa, bufb = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
        for k in range(iters):
            a.local_step_with_grads(to_dev(host[k][:16]))
            b.local_step_with_grads(to_dev(host[k][16:]))
            if (k + 1) % tau == 0:
                _sync_two(a, b, bufa, bufb)
                assert a.summed_floats == (P if fusion else 0) and b.summed_floats == a.summed_floats
        states[fusion] = (a.state(), b.state())
        a.close()
        b.close()
    for sa, sb in zip(states[True], states[False]):
        for u, w in zip(sa, sb):
            assert np.array_equal(u, w)
    (xa, za, va), (xb, zb, vb) = states[True]
    assert np.array_equal(za, zb) and np.array_equal(va, vb)
    got = [xa[i] for i in range(16)] + [xb[i] for i in range(8)] + [za]
    want = [st.x[i] for i in range(m)] + [st.z]
    assert max_rel_err(got, want) <= 1e-5


def test_shards_of_a_tensor_core_model_sum_their_workers_inside_the_sync_step_launch():
    """Hidden layers on the tensor cores, workers split 8 + 8: each shard's sync-step
    weight-gradient launch adds up its own workers' weight matrices, the partial-sum buffer
    handed to the exchange is the same to the bit as with the worker-mean kernel, and the
    trajectory is the oracle's 16-worker one."""
    from paper_2002_09539_b200 import OverlapLocalSGD
    dims, m, n, batch, tau, iters = [128, 256, 128, 10], 16, 96, 64, 2, 6
    X, y = si.mixture_data(23, m, n, dims[0])
    x0 = si.model_init(23, "mlp", dims)
    kw = dict(tau=tau, batch=batch, gamma=0.02, alpha=0.6, beta=0.9, mu=0.9, seed=23)
    st, lo, _ = runner.run_model("mlp", dims, X, y, x0, m=m, iters=iters, bf16_operands=True, **kw)
    weights = dims[1] * dims[0] + dims[2] * dims[1]
    got = {}
    for fusion in (True, False):
        sh = [OverlapLocalSGD("mlp", dims=dims, gemm_bf16=1, x0=x0, X=to_dev(X[o:o + 8]),
                              y=to_dev(y[o:o + 8]), m=8, worker_offset=o, m_total=m, **kw)
              for o in (0, 8)]
        for ctx in sh:
            ctx.set_anchor_fusion(fusion)
        rows = sh[0].lib.olsgd_row_floats(sh[0].ctx)
        bufs = [torch.zeros(rows, device="cuda") for _ in sh]
        loss = [torch.zeros((iters, 8), device="cuda") for _ in sh]
        totals = []
        for k in range(iters):
            for ctx, l in zip(sh, loss):
                ctx.local_step(l[k])
            if (k + 1) % tau == 0:
                totals.append(_sync_two(sh[0], sh[1], bufs[0], bufs[1]).cpu().numpy())
                assert all(ctx.summed_floats == (weights if fusion else 0) for ctx in sh)
        xs = [ctx.get_params(i).copy() for ctx in sh for i in range(8)]
        got[fusion] = (xs, sh[0].get_params(-1).copy(), sh[1].get_params(-1).copy(), totals,
                       np.concatenate([l.cpu().numpy() for l in loss], axis=1))
        for ctx in sh:
            ctx.close()
    on, off = got[True], got[False]
    assert all(np.array_equal(a, b) for a, b in zip(on[0], off[0]))
    assert np.array_equal(on[1], off[1]) and np.array_equal(on[1], on[2])
    assert all(np.array_equal(a, b) for a, b in zip(on[3], off[3]))
    assert np.array_equal(on[4], off[4])
    want = [st.x[i] for i in range(m)] + [st.z]
    assert max_rel_err(on[0] + [on[1]], want) <= 5e-3
    assert np.abs(on[4] - lo).max() <= 2e-2 * np.abs(lo).max()


def test_two_shards_of_a_model_draw_the_global_minibatches():
    from paper_2002_09539_b200 import OverlapLocalSGD
    m, n, d, C, batch, tau, iters = 4, 80, 96, 10, 16, 2, 4
    X, y = si.mixture_data(6, m, n, d)
    x0 = (0.05 * np.random.default_rng(6).standard_normal(d * C + C)).astype(np.float32)
    kw = dict(tau=tau, batch=batch, gamma=0.1, alpha=0.5, beta=0.7, mu=0.9, seed=6)
    st, lo, _ = runner.run_model("softmax", [d, C], X, y, x0, m=m, iters=iters, **kw)
    sh = [OverlapLocalSGD("softmax", dims=[d, C], x0=x0, X=to_dev(X[o:o + 2]), y=to_dev(y[o:o + 2]),
                          m=2, worker_offset=o, m_total=m, **kw) for o in (0, 2)]
    for o, ctx in zip((0, 2), sh):
        assert np.array_equal(ctx.get_indices(3), sampling.minibatch_indices(6, m, 3, batch, n)[o:o + 2])
    rows = sh[0].lib.olsgd_row_floats(sh[0].ctx)
    bufs = [torch.zeros(rows, device="cuda") for _ in sh]
    loss = [torch.zeros((iters, 2), device="cuda") for _ in sh]
    for k in range(iters):
        for ctx, l in zip(sh, loss):
            ctx.local_step(l[k])
        if (k + 1) % tau == 0:
            _sync_two(sh[0], sh[1], bufs[0], bufs[1])
    got = [ctx.get_params(i).copy() for ctx in sh for i in range(2)] + [sh[0].get_params(-1).copy()]
    want = [st.x[i] for i in range(m)] + [st.z]
    assert max_rel_err(got, want) <= 1e-5
    lg = np.concatenate([l.cpu().numpy() for l in loss], axis=1)
    assert np.abs(lg - lo).max() <= 2e-5 * np.abs(lo).max()
