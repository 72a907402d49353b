"""NumPy twin of the sequential simulator, for tiny cases -- TEST INFRASTRUCTURE.

Same steps, same order, written independently of the C file so that each checks the other:
the mixing flow of Eq. (dynamic) in closed form (Algorithm 1's matrix exponential), the
gradient jump and the pairwise jump."""
from __future__ import annotations

import numpy as np


class NumpySim:
    def __init__(self, x0, eta, alpha, alpha_tilde, gamma, grads=None, xt0=None, t0=None, variant=0):
        self.X = np.array(x0, dtype=np.float64)
        self.Xt = self.X.copy() if xt0 is None else np.array(xt0, dtype=np.float64)
        self.n, self.d = self.X.shape
        self.t = np.zeros(self.n) if t0 is None else np.array(t0, dtype=np.float64)
        self.G = None if grads is None else np.array(grads, dtype=np.float64)
        self.eta, self.alpha, self.alpha_tilde, self.gamma = float(eta), float(alpha), float(alpha_tilde), float(gamma)
        self.variant = int(variant)

    def mix(self, w, t):
        """exp((t - t_w) [[-eta, eta],[eta, -eta]]) applied to (x_w, x~_w)."""
        dt = t - self.t[w]
        if dt < 0:
            raise ValueError("event before the worker's last event")
        e = np.exp(-2.0 * self.eta * dt)
        m00 = 0.5 * (1.0 + e)
        m01 = 0.5 * (1.0 - e)
        x, xt = self.X[w].copy(), self.Xt[w].copy()
        self.X[w] = m00 * x + m01 * xt
        self.Xt[w] = m01 * x + m00 * xt
        self.t[w] = t

    def grad_event(self, t, i, s):
        if self.variant == 2:  # Eq. (baselinedynamic): x alone, no flow
            self.X[i] -= self.gamma * self.G[s]
            self.t[i] = t
            return
        self.mix(i, t)
        self.X[i] -= self.gamma * self.G[s]
        self.Xt[i] -= self.gamma * self.G[s]

    def comm_event(self, t, i, j):
        if self.variant == 2:
            m = self.X[i] - self.X[j]
            self.X[i] -= self.alpha * m
            self.X[j] += self.alpha * m
            self.t[i] = self.t[j] = t
            return
        if self.variant == 1:
            m = self.X[i] - self.X[j]
            self.mix(i, t)
            self.mix(j, t)
        else:
            self.mix(i, t)
            self.mix(j, t)
            m = self.X[i] - self.X[j]
        self.X[i] -= self.alpha * m
        self.Xt[i] -= self.alpha_tilde * m
        self.X[j] += self.alpha * m
        self.Xt[j] += self.alpha_tilde * m

    def apply(self, times, wi, wj, slot):
        for t, i, j, s in zip(times, wi, wj, slot):
            if j < 0:
                self.grad_event(float(t), int(i), int(s))
            else:
                self.comm_event(float(t), int(i), int(j))

    def consensus(self):
        xbar = self.X.mean(axis=0, keepdims=True)
        return float(((self.X - xbar) ** 2).sum())
