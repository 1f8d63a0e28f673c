"""Loss ell(x; s) and minibatch gradient g_i(x; xi) of the three model families.

The paper leaves the model open (Section 2, Eq. 1: any per-sample loss
ell(x; s)); these are the families of the benchmark configurations.  Every
function returns the MEAN loss over the rows it is given and the gradient of
that mean, in fp64.

Flat parameter layout (an interface shared, by specification, with the CUDA
library's header): for each layer l in order, the weight matrix W_l stored
row-major as [out][in], followed by its bias b_l [out].  Linear regression has
one weight vector w [d] and no bias.

`bf16_operands=True` rounds the operands of every matrix product (inputs,
weights, hidden activations, back-propagated pre-activation gradients) to
bfloat16 with round-to-nearest-even and keeps everything else in fp64.  It is a
debugging aid for the bf16 tensor-core path; the default is exact fp64.

This is test infrastructure (see the package docstring).
"""
import numpy as np


def round_bf16(a):
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even)."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(a))


def n_params(kind, dims):
    if kind == "linreg":
        return dims[0]
    return sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))


def unpack(dims, params):
    """Split a flat parameter vector into [(W_l, b_l)] views."""
    out, off = [], 0
    for l in range(len(dims) - 1):
        fan_in, fan_out = dims[l], dims[l + 1]
        W = params[off:off + fan_out * fan_in].reshape(fan_out, fan_in)
        off += fan_out * fan_in
        b = params[off:off + fan_out]
        off += fan_out
        out.append((W, b))
    assert off == params.size
    return out


def linreg_loss_grad(w, X, y):
    """loss = (1/2B) sum_s (x_s . w - y_s)^2 ;  grad = X^T (X w - y) / B."""
    w = np.asarray(w, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    r = X @ w - y
    B = X.shape[0]
    return 0.5 * float(r @ r) / B, X.T @ r / B


def _log_softmax(logits):
    shifted = logits - logits.max(axis=1, keepdims=True)
    return shifted - np.log(np.exp(shifted).sum(axis=1, keepdims=True))


def mlp_loss_grad(dims, params, X, labels, bf16_operands=False, want_grad=True):
    """ReLU multilayer perceptron with mean cross-entropy on the last layer.

    dims = [d_in, h_1, ..., n_classes]; two entries give softmax regression.
    """
    q = round_bf16 if bf16_operands else (lambda a: a)
    params = np.asarray(params, dtype=np.float64)
    layers = unpack(dims, params)
    L = len(layers)
    B = X.shape[0]
    labels = np.asarray(labels).astype(np.int64)

    acts = [q(np.asarray(X, dtype=np.float64))]       # operand of layer 0
    for l, (W, b) in enumerate(layers):
        a = acts[-1] @ q(W).T + b
        if l < L - 1:
            a = q(np.maximum(a, 0.0))                 # hidden activation
        acts.append(a)
    logp = _log_softmax(acts[-1])
    loss = -float(logp[np.arange(B), labels].sum()) / B
    if not want_grad:
        return loss, None

    grad = np.empty_like(params)
    gviews = unpack(dims, grad)
    delta = np.exp(logp)
    delta[np.arange(B), labels] -= 1.0
    delta /= B                                        # d loss / d logits
    for l in range(L - 1, -1, -1):
        W, _ = layers[l]
        gW, gb = gviews[l]
        gb[:] = delta.sum(axis=0)
        dq = q(delta)
        gW[:] = dq.T @ acts[l]
        if l > 0:
            delta = (dq @ q(W)) * (acts[l] > 0.0)
    return loss, grad


def loss_grad(kind, dims, params, X, y, bf16_operands=False):
    if kind == "linreg":
        return linreg_loss_grad(params, X, y)
    return mlp_loss_grad(dims, params, X, y, bf16_operands=bf16_operands)


def full_objective(kind, dims, params, X_all, y_all, bf16_operands=False):
    """F(x) of Eq. 1 with D_i the empirical distribution of worker i's rows:
    the mean over workers of the mean loss on that worker's whole partition."""
    total = 0.0
    for Xi, yi in zip(X_all, y_all):
        if kind == "linreg":
            total += linreg_loss_grad(params, Xi, yi)[0]
        else:
            total += mlp_loss_grad(dims, params, Xi, yi, bf16_operands, want_grad=False)[0]
    return total / len(X_all)
