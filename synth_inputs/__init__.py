"""Seeded synthetic inputs and the benchmark configuration table.

This module is the only code shared by the CUDA path and the CPU oracle.  It
produces arrays (datasets, initial weights, external gradients) from a seed
with numpy's PCG64 generator and holds none of the method's arithmetic: no
update rule, no loss, no gradient, no minibatch sampling.

Stand-in statement: the paper trains ResNet-18 on CIFAR-10 with 16 workers and
128 samples per worker per step, IID and class-skewed.  Neither the dataset nor
the network is used here.  The synthetic Gaussian mixture below keeps the
shapes that matter to the hot path (3072 = 32*32*3 input features, ten
classes, per-worker partitions, IID or two-classes-per-worker).
"""
import numpy as np

N_CLASSES = 10

# Hyper-parameters of the five benchmark configurations.  `beta` is the
# paper's anchor momentum factor, `mu` the local Nesterov factor; the momentum
# configurations quote one number and it is used for both.
CONFIGS = {
    "c1": dict(kind="linreg", dims=[64], m=4, n=1024, batch=32, tau=2, gamma=0.05,
               alpha=0.5, beta=0.0, mu=0.0, iters=100, gemm_bf16=0, non_iid=False),
    "c2": dict(kind="softmax", dims=[3072, 10], m=16, n=5000, batch=128, tau=2, gamma=0.1,
               alpha=0.6, beta=0.0, mu=0.0, iters=500, gemm_bf16=0, non_iid=False),
    "c3": dict(kind="mlp", dims=[3072, 1024, 1024, 10], m=16, n=5000, batch=128, tau=2,
               gamma=0.05, alpha=0.6, beta=0.9, mu=0.9, iters=1000, gemm_bf16=1,
               non_iid=False),
    "c4": dict(kind="mlp", dims=[3072, 512, 10], m=64, n=5000, batch=64, tau=8,
               gamma=0.05, alpha=0.5, beta=0.9, mu=0.9, iters=800, gemm_bf16=1,
               non_iid=True),
    "c5": dict(kind="flat", P=[1_000_000, 10_000_000, 50_000_000], m=[8, 16, 64], tau=4,
               gamma=0.05, alpha=0.5, beta=0.9, mu=0.9, grad_std=0.1),
}


def _rng(seed, tag):
    return np.random.Generator(np.random.PCG64([int(seed), int(tag)]))


def linreg_data(seed, m, n, d):
    """X[m][n][d] ~ N(0,1); one shared w* ~ N(0,1); y = X w* + N(0, 0.1^2)."""
    rng = _rng(seed, 101)
    w_star = rng.standard_normal(d)
    X = rng.standard_normal((m, n, d)).astype(np.float32)
    noise = 0.1 * rng.standard_normal((m, n))
    y = (X.astype(np.float64) @ w_star + noise).astype(np.float32)
    return X, y, w_star


def mixture_means(seed, d):
    """Ten class means, each ~ N(0, I/d)."""
    return (_rng(seed, 201).standard_normal((N_CLASSES, d)) / np.sqrt(d)).astype(np.float32)


def mixture_data(seed, m, n, d, class_table=None):
    """Per-worker samples mean[label] + N(0, I).

    class_table None: labels uniform over the ten classes (IID workers).
    class_table [m][c]: sample s of worker i has label class_table[i][s % c]
    (equal shares of the worker's c classes).
    Returns X [m][n][d] float32 and labels [m][n] int32.
    """
    means = mixture_means(seed, d)
    X = np.empty((m, n, d), dtype=np.float32)
    y = np.empty((m, n), dtype=np.int32)
    for i in range(m):
        rng = _rng(seed, 1000 + i)
        if class_table is None:
            y[i] = rng.integers(0, N_CLASSES, size=n, dtype=np.int32)
        else:
            row = np.asarray(class_table[i], dtype=np.int32)
            y[i] = row[np.arange(n) % row.size]
        X[i] = rng.standard_normal((n, d), dtype=np.float32)
        X[i] += means[y[i]]
    return X, y


def model_init(seed, kind, dims):
    """Flat initial parameters x0 (float32) in the library's layout.

    Linear and softmax regression start at zero; MLP weights ~ N(0, 2/fan_in),
    biases zero.
    """
    if kind == "linreg":
        return np.zeros(dims[0], dtype=np.float32)
    rng = _rng(seed, 301)
    parts = []
    for l in range(len(dims) - 1):
        fan_in, fan_out = dims[l], dims[l + 1]
        if kind == "softmax":
            W = np.zeros((fan_out, fan_in), dtype=np.float32)
        else:
            W = (rng.standard_normal((fan_out, fan_in)) * np.sqrt(2.0 / fan_in)).astype(np.float32)
        parts += [W.ravel(), np.zeros(fan_out, dtype=np.float32)]
    return np.concatenate(parts)


def flat_init(seed, P):
    """x0 ~ N(0,1) for the flat-parameter (external gradient) workload."""
    return _rng(seed, 401).standard_normal(P, dtype=np.float32)


def flat_grads(seed, k, m, P, std=0.1):
    """External gradients of iteration k, [m][P] ~ N(0, std^2), float32."""
    return (std * _rng(seed, 500000 + k).standard_normal((m, P), dtype=np.float32)).astype(np.float32)
