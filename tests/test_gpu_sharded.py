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
