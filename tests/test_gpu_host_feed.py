"""Host-fed steps (olsgd_local_step_host, olsgd_local_step_host_bf16) against the device-sampled
step: the same minibatch rows, taken on the host with the indices the index rule gives, must
produce the same bits."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _make(kind, dims, gemm, m, n, batch, tau, seed=5):
    from paper_2002_09539_b200 import OverlapLocalSGD
    X, y = si.mixture_data(seed, m, n, dims[0])
    y = (y % dims[-1]).astype(np.int32)
    x0 = si.model_init(seed, kind, dims)
    kw = dict(m=m, tau=tau, batch=batch, gamma=0.05, alpha=0.6, beta=0.9, mu=0.9, seed=seed,
              dims=dims, gemm_bf16=gemm, x0=x0)

    def new():
        return OverlapLocalSGD(kind, X=torch.from_numpy(X).cuda(), y=torch.from_numpy(y).cuda(), **kw)
    return X, y, new


def _host_fed_run(opt, X, y, iters, dtype, ref):
    """Feeds the rows that `ref` (a context at iteration 0 with the same seed) would draw."""
    m, B = opt.m, opt.batch
    losses = torch.zeros((iters, m), dtype=torch.float32).pin_memory()
    keep = []
    for k in range(iters):
        idx = ref.get_indices(k)
        idx = idx.cpu().numpy() if hasattr(idx, "cpu") else np.asarray(idx)
        Xb = torch.from_numpy(np.stack([X[i][idx[i]] for i in range(m)])).to(dtype).pin_memory()
        yb = torch.from_numpy(np.stack([y[i][idx[i]] for i in range(m)])).pin_memory()
        keep.append((Xb, yb))
        opt.local_step_host(Xb, yb, losses[k])
        if opt.iteration % opt.tau == 0:
            opt.period_sync()
    opt.join()
    return losses.numpy().copy()


CASES = [("softmax", [100, 7], 0, 3, 50, 20, 2),
         ("mlp", [128, 256, 128, 10], 1, 2, 96, 64, 2),
         ("mlp", [192, 128, 7], 3, 3, 80, 128, 3),
         ("mlp", [64, 128, 10], 2, 2, 40, 24, 2)]


@pytest.mark.parametrize("kind,dims,gemm,m,n,batch,tau", CASES)
def test_host_fed_steps_give_the_bits_of_device_sampled_steps(kind, dims, gemm, m, n, batch, tau):
    iters = 2 * tau + 1
    X, y, new = _make(kind, dims, gemm, m, n, batch, tau)
    dev, host = new(), new()
    loss_d = torch.zeros((iters, m), device="cuda")
    for k in range(iters):
        dev.local_step(loss_d[k])
        if dev.iteration % tau == 0:
            dev.period_sync()
    ref = new()
    loss_h = _host_fed_run(host, X, y, iters, torch.float32, ref)
    xd, zd, _ = dev.state()
    xh, zh, _ = host.state()
    assert np.array_equal(xd, xh) and np.array_equal(zd, zh)
    assert np.array_equal(loss_d.cpu().numpy(), loss_h)
    for o in (dev, host, ref):
        o.close()


@pytest.mark.parametrize("kind,dims,gemm,m,n,batch,tau", CASES[1:])
def test_bf16_host_rows_give_the_bits_of_fp32_host_rows(kind, dims, gemm, m, n, batch, tau):
    iters = 2 * tau + 1
    X, y, new = _make(kind, dims, gemm, m, n, batch, tau)
    a, b, ref = new(), new(), new()
    loss_a = _host_fed_run(a, X, y, iters, torch.float32, ref)
    loss_b = _host_fed_run(b, X, y, iters, torch.bfloat16, ref)
    xa, za, _ = a.state()
    xb, zb, _ = b.state()
    assert np.array_equal(xa, xb) and np.array_equal(za, zb)
    assert np.array_equal(loss_a, loss_b)
    for o in (a, b, ref):
        o.close()


def test_bf16_host_rows_are_refused_by_fp32_models():
    from paper_2002_09539_b200.binding import OlsgdError
    X, y, new = _make("softmax", [100, 7], 0, 2, 30, 8, 2)
    opt = new()
    Xb = torch.zeros((2, 8, 100), dtype=torch.bfloat16).pin_memory()
    yb = torch.zeros((2, 8), dtype=torch.int32).pin_memory()
    with pytest.raises(OlsgdError):
        opt.local_step_host(Xb, yb)
    assert opt.iteration == 0
    opt.close()


def _mixed_sequence(opt, ref, X, y, dtype):
    """Device-sampled steps, host-fed steps, a long run (captured graph where the streams
    allow one), a jump of the iteration counter and more steps, in one context."""
    m, tau = opt.m, opt.tau
    keep = []

    def sync():
        if opt.iteration % tau == 0:
            opt.period_sync()

    def device_steps(count):
        for _ in range(count):
            opt.local_step()
            sync()

    def host_steps(count):
        for _ in range(count):
            idx = ref.get_indices(opt.iteration)
            Xb = torch.from_numpy(np.stack([X[i][idx[i]] for i in range(m)])).to(dtype).pin_memory()
            yb = torch.from_numpy(np.stack([y[i][idx[i]] for i in range(m)])).pin_memory()
            keep.append((Xb, yb))
            opt.local_step_host(Xb, yb)
            sync()

    device_steps(3)
    host_steps(2)
    device_steps(1)
    host_steps(1)
    device_steps(tau - opt.iteration % tau if opt.iteration % tau else 0)   # to a period boundary
    opt.run(40)
    host_steps(1)
    device_steps(2 * tau - 1)
    opt.join()
    opt.set_iteration(4 * tau)
    device_steps(3)
    opt.run(7)
    opt.join()
    return opt.state()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_staging_ahead_gives_the_bits_of_serial_streams(dtype):
    """With overlap (rows of the next iteration staged on the context's own stream, host rows
    staged on the copy stream, captured graphs) and with one serial stream the same mixed
    sequence of calls must end in the same bits."""
    from paper_2002_09539_b200 import OverlapLocalSGD
    dims, m, n, batch, tau, seed = [128, 256, 128, 10], 3, 96, 64, 2, 9
    X, y = si.mixture_data(seed, m, n, dims[0])
    y = (y % dims[-1]).astype(np.int32)
    x0 = si.model_init(seed, "mlp", dims)
    kw = dict(m=m, tau=tau, batch=batch, gamma=0.05, alpha=0.6, beta=0.9, mu=0.9, seed=seed,
              dims=dims, gemm_bf16=1, x0=x0)
    states = []
    for overlap in (True, False):
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            new = lambda: OverlapLocalSGD("mlp", X=torch.from_numpy(X).cuda(),
                                          y=torch.from_numpy(y).cuda(), overlap=overlap, **kw)
            opt, ref = new(), new()
            states.append(_mixed_sequence(opt, ref, X, y, dtype))
            if overlap:
                assert opt.graph_replays > 0
            opt.close()
            ref.close()
        stream.synchronize()
    for a, b in zip(states[0], states[1]):
        assert np.array_equal(a, b)
