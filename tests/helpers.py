"""Shared helpers of the GPU parity tests (not collected by pytest)."""
import numpy as np
import torch


def max_rel_err(got, want):
    """max over tensors T of ||T_gpu - T_oracle||_inf / ||T_oracle||_inf, the
    'max relative parameter error' of the acceptance bar; got/want are lists."""
    worst = 0.0
    for g, w in zip(got, want):
        g = np.asarray(g, dtype=np.float64)
        w = np.asarray(w, dtype=np.float64)
        denom = np.abs(w).max()
        err = np.abs(g - w).max()
        worst = max(worst, err / denom if denom > 0 else err)
    return worst


def state_err(opt, st):
    """Compare a GPU context with an oracle state: x_1..x_m and z."""
    x, z, v = opt.state()
    tensors_g = [x[i] for i in range(opt.m)] + [z]
    tensors_o = [st.x[i] for i in range(opt.m)] + [st.z]
    return max_rel_err(tensors_g, tensors_o)


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()
