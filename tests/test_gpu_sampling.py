"""S0/S1 on the device against the oracle: bit-exact integers."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import synth_inputs as si
from oracle import sampling
from helpers import to_dev


@pytest.mark.parametrize("seed,m,batch,n", [(0, 16, 128, 5000), (0, 4, 32, 1024),
                                            (0xDEADBEEFCAFEF00D, 64, 64, 5000),
                                            (7, 3, 13, 17), (9, 1, 1, 1), (3, 5, 130, 2**31 - 1)])
def test_minibatch_indices_bit_exact(seed, m, batch, n):
    d = 8
    n_alloc = min(n, 64)    # only olsgd_get_indices is called: no data row is ever read
    X = torch.zeros((m, n_alloc, d), device="cuda")
    y = torch.zeros((m, n_alloc), device="cuda")
    import ctypes as C
    from paper_2002_09539_b200 import binding
    lib = binding.load_library()
    spec = binding._spec("linreg", [d])
    hp = binding._HParams(m, 2, batch, 0, 0.1, 0.5, 0.0, 0.0, seed)
    nbytes = C.c_size_t()
    assert lib.olsgd_workspace_bytes(C.byref(spec), C.byref(hp), C.byref(nbytes)) == 0
    ws = torch.empty(nbytes.value + 256, dtype=torch.uint8, device="cuda")
    ptr = (ws.data_ptr() + 255) // 256 * 256
    data = binding._Data(X.data_ptr(), y.data_ptr(), n)
    x0 = torch.zeros(d, device="cuda")
    ctx = C.c_void_p()
    s = torch.cuda.current_stream().cuda_stream
    assert lib.olsgd_init(C.byref(ctx), C.byref(spec), C.byref(hp), C.byref(data), x0.data_ptr(),
                          ptr, nbytes.value, s, s) == 0
    for k in (0, 1, 2, 999, 2**31 + 5):
        out = torch.empty((m, batch), dtype=torch.int32)
        assert lib.olsgd_get_indices(ctx, k, out.data_ptr()) == 0
        want = sampling.minibatch_indices(seed, m, k, batch, n)
        assert np.array_equal(out.numpy(), want), k
    lib.olsgd_destroy(ctx)


@pytest.mark.parametrize("seed,m", [(0, 64), (0, 1), (5, 4), (5, 5), (5, 6), (2**63 + 11, 1000)])
def test_class_pairs_bit_exact(seed, m):
    from paper_2002_09539_b200 import class_pairs
    want = sampling.class_pairs(seed, m)
    got_dev = class_pairs(seed, m, device="cuda").cpu().numpy()
    got_host = class_pairs(seed, m, device="cpu").numpy()
    assert np.array_equal(got_dev, want)
    assert np.array_equal(got_host, want)


@pytest.mark.parametrize("seed,m,batch,n,offset", [(0, 4, 32, 1000, 0), (7, 3, 13, 17, 0),
                                                   (2**40 + 3, 2, 64, 5000, 6), (1, 2, 8, 1, 0),
                                                   (5, 2, 16, 1024, 0)])
def test_epoch_rule_indices_bit_exact(seed, m, batch, n, offset):
    from paper_2002_09539_b200 import OverlapLocalSGD
    d = 8
    X = torch.zeros((m, n, d), device="cuda")
    y = torch.zeros((m, n), device="cuda")
    opt = OverlapLocalSGD("linreg", m=m, tau=2, gamma=0.1, alpha=0.5, batch=batch, seed=seed,
                          dims=[d], x0=np.zeros(d, np.float32), X=X, y=y, epoch_sampling=True,
                          worker_offset=offset, m_total=offset + m)
    for k in (0, 1, 2, n // batch, 3 * n + 1, 12345):
        want = sampling.minibatch_indices_epoch(seed, m, k, batch, n, worker_offset=offset)
        assert np.array_equal(opt.get_indices(k), want), k
