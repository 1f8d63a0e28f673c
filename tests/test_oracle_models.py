"""Pins for oracle.models: finite differences, textbook special cases, a
library routine for the least-squares solution and for bf16 rounding."""
import numpy as np
import pytest
import torch

from oracle import models


def _fd(f, x, eps=1e-6):
    g = np.zeros_like(x)
    for j in range(x.size):
        xp, xm = x.copy(), x.copy()
        xp[j] += eps
        xm[j] -= eps
        g[j] = (f(xp) - f(xm)) / (2 * eps)
    return g


def test_linreg_gradient_finite_difference():
    rng = np.random.default_rng(0)
    X, y, w = rng.standard_normal((5, 8)), rng.standard_normal(5), rng.standard_normal(8)
    loss, g = models.linreg_loss_grad(w, X, y)
    assert loss == pytest.approx(0.5 * np.mean((X @ w - y) ** 2), rel=1e-14)
    fd = _fd(lambda p: models.linreg_loss_grad(p, X, y)[0], w)
    assert np.allclose(g, fd, rtol=1e-7, atol=1e-9)


def test_linreg_full_batch_descent_reaches_normal_equations():
    rng = np.random.default_rng(1)
    X, y = rng.standard_normal((40, 6)), rng.standard_normal(40)
    w = np.zeros(6)
    for _ in range(4000):
        w = w - 0.1 * models.linreg_loss_grad(w, X, y)[1]
    assert np.allclose(w, np.linalg.lstsq(X, y, rcond=None)[0], atol=1e-10)


@pytest.mark.parametrize("dims", [[6, 4], [5, 7, 3], [4, 6, 5, 3]])
def test_mlp_gradient_finite_difference(dims):
    rng = np.random.default_rng(2)
    P = models.n_params("mlp", dims)
    x = rng.standard_normal(P) * 0.5
    X = rng.standard_normal((6, dims[0]))
    lab = rng.integers(0, dims[-1], size=6)
    loss, g = models.mlp_loss_grad(dims, x, X, lab)
    fd = _fd(lambda p: models.mlp_loss_grad(dims, p, X, lab, want_grad=False)[0], x)
    assert np.allclose(g, fd, rtol=1e-6, atol=1e-8), np.abs(g - fd).max()


def test_softmax_special_cases():
    # zero weights: uniform prediction, loss = ln C, dW = (1/C - onehot)^T X / B
    dims = [5, 10]
    rng = np.random.default_rng(3)
    X, lab = rng.standard_normal((7, 5)), rng.integers(0, 10, 7)
    loss, g = models.mlp_loss_grad(dims, np.zeros(60), X, lab)
    assert loss == pytest.approx(np.log(10.0), rel=1e-14)
    onehot = np.eye(10)[lab]
    (gW, gb), = models.unpack(dims, g)
    assert np.allclose(gW, (0.1 - onehot).T @ X / 7)
    assert np.allclose(gb, (0.1 - onehot).sum(0) / 7)
    # two classes reduce to logistic regression on the logit difference
    dims2 = [5, 2]
    x = rng.standard_normal(12)
    lab2 = rng.integers(0, 2, 7)
    (W, b), = models.unpack(dims2, x)
    t = X @ (W[1] - W[0]) + (b[1] - b[0])
    want = np.mean(np.log1p(np.exp(-np.where(lab2 == 1, t, -t))))
    assert models.mlp_loss_grad(dims2, x, X, lab2)[0] == pytest.approx(want, rel=1e-12)


def test_softmax_is_shift_invariant_and_stable():
    dims = [3, 4]
    x = np.zeros(16)
    (W, b), = models.unpack(dims, x)
    b[:] = [1000.0, 999.0, 998.0, 0.0]          # would overflow without max-subtraction
    X, lab = np.ones((2, 3)), np.array([0, 1])
    loss, g = models.mlp_loss_grad(dims, x, X, lab)
    b2 = x.copy()
    models.unpack(dims, b2)[0][1][:] -= 1000.0
    loss2, g2 = models.mlp_loss_grad(dims, b2, X, lab)
    assert np.isfinite(loss) and loss == pytest.approx(loss2, rel=1e-12)
    assert np.allclose(g, g2)


def test_layout_is_weights_then_bias_per_layer():
    dims = [3, 2, 4]
    x = np.arange(models.n_params("mlp", dims), dtype=np.float64)
    (W0, b0), (W1, b1) = models.unpack(dims, x)
    assert W0.shape == (2, 3) and W0[1, 0] == 3 and list(b0) == [6, 7]
    assert W1.shape == (4, 2) and W1[0, 0] == 8 and list(b1) == [16, 17, 18, 19]
    assert models.n_params("linreg", [64]) == 64
    assert models.n_params("softmax", [3072, 10]) == 30730
    assert models.n_params("mlp", [3072, 1024, 1024, 10]) == 4206602
    assert models.n_params("mlp", [3072, 512, 10]) == 1578506


def test_bf16_rounding_matches_library_cast():
    rng = np.random.default_rng(4)
    a = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        # exact ties between two bf16 neighbours
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 0.0])])
    a = a.astype(np.float32)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(models.round_bf16(a), want)


def test_bf16_mode_is_close_to_exact_and_not_identical():
    dims = [16, 12, 5]
    rng = np.random.default_rng(6)
    x = rng.standard_normal(models.n_params("mlp", dims)) * 0.3
    X, lab = rng.standard_normal((8, 16)), rng.integers(0, 5, 8)
    l0, g0 = models.mlp_loss_grad(dims, x, X, lab)
    l1, g1 = models.mlp_loss_grad(dims, x, X, lab, bf16_operands=True)
    assert l0 != l1 and abs(l0 - l1) < 2e-2 * abs(l0)
    assert np.abs(g0 - g1).max() < 2e-2 * np.abs(g0).max()


def test_bf16_rounding_points_worked_by_hand():
    """Which operands `bf16_operands=True` rounds, pinned on a 2-2-2 network whose values sit on
    bf16 ties, with the expected loss and gradient worked out by hand below (no oracle routine
    is called to produce them).  bf16 keeps 8 significant bits; with e = 2^-8 the representable
    numbers are e apart in [0.5, 1), 2e apart in [1, 2), 4e in [2, 4), and a tie goes to the
    neighbour whose last kept bit is 0.

    Roundings used:  1+e -> 1,  1+3e -> 1+4e,  2+2e -> 2,  0.5+e/2 would go to 0.5 and 64.125
    to 64 (but biases are NOT rounded).

    Forward.  q(X) = [[-1, 1], [1+4e, -0.5], [.75, .25]],  q(W1) = [[1, .5], [1+4e, -1]],
    b1 = [0.5+e/2, 1].
      sample 0: unit 0 = -1 + .5 + .5 + e/2 = e/2;                unit 1 = -(1+4e) - 1 + 1 < 0
      sample 1: unit 0 = (1+4e) - .25 + .5 + e/2 = 1.25 + 4.5e;   unit 1 = (1+4e)^2 + .5 + 1
      sample 2: unit 0 = .75 + .125 + .5 + e/2 = 1.375 + e/2;     unit 1 = .75(1+4e) - .25 + 1
    rounded hidden activations: [[e/2, 0], [1.25+4e, 2.5+8e], [1.375, 1.5+4e]]
    (1.5+3e is a tie: 1.5+2e ends in an odd bit, so it goes to 1.5+4e).
    q(W2) = [[1, -(1+4e)], [3, 2]], b2 = [0, 64.125], so
      logit_1 - logit_0 = h . [2, 3+4e] + 64.125  >= 64 for every sample:
    softmax puts probability 1 (to 1e-27) on class 1.  Samples 0 and 1 carry label 0, so their
    loss is that gap; sample 2 carries label 1 and contributes 0:
      gap_0 = 2(e/2) + 64.125 = 64.125 + e
      gap_1 = 2(1.25+4e) + (2.5+8e)(3+4e) + 64.125 = 74.125 + 42e + 32e^2
      loss  = (gap_0 + gap_1) / 3.

    Backward.  d loss / d logits = [-1/3, +1/3] for samples 0 and 1, zero for sample 2.
      bias gradient of layer 2 (from the unrounded values): [-2/3, 2/3]
      D = q(1/3): 1/3 = 1.0101010 1010..b x 2^-2 rounds up to 1.0101011b x 2^-2 = 171/512
      dW2 = [-D, D]^T (h_0 + h_1) with h_0 + h_1 = [1.25 + 4.5e, 2.5 + 8e]
      into the hidden layer: D * (q(W2)[1] - q(W2)[0]) = D [2, 3+4e], masked by h > 0:
        sample 0: [2D, 0],   sample 1: [2D, D(3+4e)]
      bias gradient of layer 1 (unrounded): [4D, D(3+4e)] = [171/128, 33003/32768]
      rounded for the weight gradient: 2D = 171/256 is representable; D(3+4e) = 33003/32768,
      33003 = 10000000 11101011b rounds up to 10000001b x 2^8, i.e. 129/128
      dW1 row 0 = 2D (q(x_0) + q(x_1)) = 2D [4e, .5] = [8De, D]
      dW1 row 1 = (129/128) q(x_1) = (129/128) [1+4e, -.5].

    Leaving out any one rounding (input, weight, hidden activation, either back-propagated
    gradient), rounding a bias, or summing the bias gradient from rounded values changes the
    loss by >= 2.8e-5 relative or a gradient entry by >= 6.5e-4.
    """
    e = 2.0 ** -8
    X = np.array([[-(1 + e), 1 + e], [1 + 3 * e, -0.5], [0.75, 0.25]])
    labels = np.array([0, 0, 1])
    W1, b1 = np.array([[1 + e, 0.5], [1 + 3 * e, -1.0]]), np.array([0.5 + e / 2, 1.0])
    W2, b2 = np.array([[1 + e, -(1 + 3 * e)], [3.0, 2 + 2 * e]]), np.array([0.0, 64.125])
    params = np.concatenate([W1.ravel(), b1, W2.ravel(), b2])
    loss, g = models.mlp_loss_grad([2, 2, 2], params, X, labels, bf16_operands=True)

    D = 171.0 / 512.0
    want_loss = ((64.125 + e) + (74.125 + 42 * e + 32 * e * e)) / 3.0
    want = np.array([8 * D * e, D,                                  # dW1 row 0
                     129.0 / 128.0 * (1 + 4 * e), -129.0 / 256.0,   # dW1 row 1
                     171.0 / 128.0, 33003.0 / 32768.0,              # db1
                     -D * (1.25 + 4.5 * e), -D * (2.5 + 8 * e),     # dW2 row 0
                     D * (1.25 + 4.5 * e), D * (2.5 + 8 * e),       # dW2 row 1
                     -2.0 / 3.0, 2.0 / 3.0])                        # db2
    assert loss == pytest.approx(want_loss, rel=1e-13)
    assert np.abs(g - want).max() <= 1e-13, np.abs(g - want)
    # the same network without operand rounding is visibly different on both
    l_exact, g_exact = models.mlp_loss_grad([2, 2, 2], params, X, labels)
    assert abs(l_exact - want_loss) > 1e-5 * want_loss and np.abs(g_exact - want).max() > 1e-4


def test_full_objective_is_mean_over_workers():
    rng = np.random.default_rng(7)
    X, y, w = rng.standard_normal((3, 9, 4)), rng.standard_normal((3, 9)), rng.standard_normal(4)
    want = np.mean([0.5 * np.mean((X[i] @ w - y[i]) ** 2) for i in range(3)])
    assert models.full_objective("linreg", [4], w, X, y) == pytest.approx(want, rel=1e-14)
