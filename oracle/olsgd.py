"""Overlap-Local-SGD and its momentum variant, step by step, in fp64.

Follows Section 2 of the paper in its order and notation:

  Eq. 3   x_{k+1/2}^(i) = x_k^(i) - gamma * g_i(x_k^(i); xi_k^(i))
  Eq. 4   x_{k+1}^(i)   = x_{k+1/2}^(i) - alpha * (x_{k+1/2}^(i) - z_k)
                           when (k+1) mod tau == 0, else x_{k+1/2}^(i)
  Eq. 5   z_{k+1}       = (1/m) sum_i x_{k+1}^(i)
                           when (k+1) mod tau == 0, else z_k
  Eq. 10  v_{k+1}       = beta * v_k + ((1/m) sum_i x_{k+1}^(i) - z_k)
  Eq. 11  z_{k+1}       = z_k + v_{k+1}          (both only on sync steps)

and, as a second statement of the same update (Section 2, "Matrix-Form Update
Rule"):

  Eq. 6-7 X_k = [x^(1), ..., x^(m), z],  G_k = [g_1, ..., g_m, 0]
  Eq. 8   X_{k+1} = (X_k - gamma * G_k) W_k
  Eq. 9   W_k = [[(1-alpha) I, (1-alpha) 1/m], [alpha 1^T, alpha]] on sync
          steps, the identity otherwise.

Readings where the paper is silent:
  * all models start equal, x_0^(i) = z_0 (Theorem 1's condition); the
    momentum buffers u_i and v start at zero;
  * "common Nesterov momentum" on the local step is the usual deep-learning
    form u <- mu*u + g, x <- x - gamma*(g + mu*u); the buffer is fed by local
    gradients only and is never pulled, averaged or reset;
  * iterations are 0-based, so the first sync happens when k + 1 == tau;
  * the anchor used by the pull-back at the end of a period is the one
    produced at the end of the previous period (the paper's remark after
    Eq. 5), which is what evaluating Eq. 4 before Eq. 5 gives.

This is test infrastructure (see the package docstring).
"""
import numpy as np


class OverlapLocalSGD:
    """State (x_1..x_m, u_1..u_m, z, v, k) and one iteration of the method."""

    def __init__(self, x0, m, tau, gamma, alpha, beta=0.0, mu=0.0):
        x0 = np.asarray(x0, dtype=np.float64)
        self.m, self.tau = int(m), int(tau)
        self.gamma, self.alpha = float(gamma), float(alpha)
        self.beta, self.mu = float(beta), float(mu)
        self.x = np.tile(x0, (self.m, 1))        # x_0^(i) = z_0 for all i
        self.u = np.zeros_like(self.x)           # local Nesterov buffers
        self.z = x0.copy()                       # anchor
        self.v = np.zeros_like(x0)               # anchor momentum buffer
        self.k = 0

    def is_sync_step(self):
        return (self.k + 1) % self.tau == 0

    def step(self, g):
        """Advance k -> k+1 given the stacked stochastic gradients g [m][P]."""
        g = np.asarray(g, dtype=np.float64)
        sync = self.is_sync_step()
        for i in range(self.m):
            # Eq. 3 (with the local Nesterov buffer when mu > 0)
            if self.mu != 0.0:
                self.u[i] = self.mu * self.u[i] + g[i]
                self.x[i] = self.x[i] - self.gamma * (g[i] + self.mu * self.u[i])
            else:
                self.x[i] = self.x[i] - self.gamma * g[i]
            # Eq. 4, against the anchor held since the previous sync
            if sync:
                self.x[i] = self.x[i] - self.alpha * (self.x[i] - self.z)
        if sync:
            s = np.zeros_like(self.z)
            for i in range(self.m):
                s += self.x[i]
            s /= self.m
            if self.beta == 0.0:
                self.v = s - self.z              # kept so that v is always defined
                self.z = s                       # Eq. 5
            else:
                self.v = self.beta * self.v + (s - self.z)   # Eq. 10
                self.z = self.z + self.v                     # Eq. 11
        self.k += 1

    def virtual_sequence(self):
        """y_k = (1-alpha) * mean_i x_k^(i) + alpha * z_k  (Appendix A)."""
        return (1.0 - self.alpha) * self.x.mean(axis=0) + self.alpha * self.z

    def mean_model(self):
        return self.x.mean(axis=0)


class LocalSGD:
    """Local SGD / periodic averaging, the baseline the paper starts from (Eq. 2):

        x_{k+1}^(i) = (1/m) sum_j [x_k^(j) - gamma g_j]   when (k+1) mod tau == 0
                    = x_k^(i) - gamma g_i                  otherwise.

    tau = 1 is fully synchronous SGD.  A local Nesterov buffer (mu > 0) is fed by local
    gradients only and is not averaged, as in OverlapLocalSGD.  `z` mirrors the last
    average so that both classes expose the same fields.
    """

    def __init__(self, x0, m, tau, gamma, mu=0.0):
        x0 = np.asarray(x0, dtype=np.float64)
        self.m, self.tau, self.gamma, self.mu = int(m), int(tau), float(gamma), float(mu)
        self.x = np.tile(x0, (self.m, 1))
        self.u = np.zeros_like(self.x)
        self.z = x0.copy()
        self.v = np.zeros_like(x0)
        self.k = 0

    def step(self, g):
        g = np.asarray(g, dtype=np.float64)
        for i in range(self.m):
            if self.mu != 0.0:
                self.u[i] = self.mu * self.u[i] + g[i]
                self.x[i] = self.x[i] - self.gamma * (g[i] + self.mu * self.u[i])
            else:
                self.x[i] = self.x[i] - self.gamma * g[i]
        if (self.k + 1) % self.tau == 0:
            s = np.zeros_like(self.z)
            for i in range(self.m):
                s += self.x[i]
            s /= self.m
            for i in range(self.m):
                self.x[i] = s
            self.z = s.copy()
        self.k += 1

    def mean_model(self):
        return self.x.mean(axis=0)


def mixing_matrix(m, alpha):
    """The sync-step W of Eq. 9, (m+1) x (m+1), column-stochastic."""
    W = np.zeros((m + 1, m + 1))
    W[:m, :m] = (1.0 - alpha) * np.eye(m)
    W[:m, m] = (1.0 - alpha) / m
    W[m, :m] = alpha
    W[m, m] = alpha
    return W


def matrix_form_step(X, G, gamma, W):
    """Eq. 8: X, G are d x (m+1) with the anchor (resp. a zero) last."""
    return (X - gamma * G) @ W

