"""Host-side choice of the quantization bit width (the MDP module of MQGrad, Section 3.3).

Two selectors, both tiny numpy programs that run on the host between launches and only call
the library through the `bits` argument:

* `SarsaBitSelector` follows the paper: MDP time step every T = 5 training iterations, state =
  [n_t, T smoothed losses] (Eq. 1), actions {keep, +1 bit} (bits never decrease), reward from
  the regression slope of the smoothed losses per millisecond (Eq. 2), a 5-10-7 Q network
  (Section 4.1) trained with SARSA (Algorithm 2) under an epsilon-greedy policy.
* `WindowQSelector` is the simpler per-iteration variant: any width in 1..8 every iteration
  from the last 10 losses, one-step Q-learning on a linear model.

Readings where the paper is silent: Q(s, a) is the network output for bit width n + a; the
discount of Algorithm 2 is 0.9 (the paper's "gamma" = 300 is the reward scale of Eq. 2); the first
state repeats the first loss; n_0 is the smallest width; a width above the range is clamped.
"""
from __future__ import annotations

import numpy as np


def smooth_losses(losses, carry, alpha):
    """Eq. 1: L~_i = alpha * L_i + (1 - alpha) * L~_{i-1}, starting from last period's L~_T."""
    out = np.empty(len(losses), np.float64)
    prev = carry
    for i, loss in enumerate(losses):
        prev = alpha * float(loss) + (1.0 - alpha) * prev
        out[i] = prev
    return out


def regression_slope(values):
    """beta of the least-squares line beta * i + b through (i, values[i-1]), i = 1..T."""
    v = np.asarray(values, np.float64)
    i = np.arange(1, v.size + 1, dtype=np.float64)
    di = i - i.mean()
    return float((di * (v - v.mean())).sum() / (di * di).sum())


def reward(smoothed, elapsed_ms, scale=300.0):
    """Eq. 2: R = -(1 / c) * beta * scale; a fast drop of the loss in little time pays most."""
    return -regression_slope(smoothed) * scale / max(float(elapsed_ms), 1e-9)


class QNetwork:
    """inputs -> hidden (ReLU) -> outputs (linear), trained by semi-gradient TD updates."""

    def __init__(self, n_in=5, n_hidden=10, n_out=7, rng=None):
        rng = rng or np.random.default_rng(0)
        self.w1 = rng.normal(0.0, 1.0 / np.sqrt(n_in), (n_hidden, n_in))
        self.b1 = np.zeros(n_hidden)
        self.w2 = rng.normal(0.0, 1.0 / np.sqrt(n_hidden), (n_out, n_hidden))
        self.b2 = np.zeros(n_out)

    def forward(self, x):
        z = self.w1 @ x + self.b1
        h = np.maximum(z, 0.0)
        return self.w2 @ h + self.b2, (x, z, h)

    def q(self, x):
        return self.forward(x)[0]

    def td_step(self, x, out_index, delta, lr):
        """v <- v + lr * delta * dQ(x)[out_index] / dv."""
        _, (x, z, h) = self.forward(x)
        dh = self.w2[out_index] * (z > 0)
        self.w2[out_index] += lr * delta * h
        self.b2[out_index] += lr * delta
        self.w1 += lr * delta * np.outer(dh, x)
        self.b1 += lr * delta * dh

    def num_parameters(self):
        return self.w1.size + self.b1.size + self.w2.size + self.b2.size


class SarsaBitSelector:
    def __init__(self, period=5, bits_min=2, bits_max=8, alpha=0.01, epsilon=0.1, lr=0.1,
                 reward_scale=300.0, discount=0.9, hidden=10, seed=0):
        self.T, self.lo, self.hi = period, bits_min, bits_max
        self.alpha, self.eps, self.lr = alpha, epsilon, lr
        self.scale, self.discount = reward_scale, discount
        self.rng = np.random.default_rng(seed)
        self.net = QNetwork(period, hidden, bits_max - bits_min + 1, self.rng)
        self.n = bits_min                   # n_t, the "most confident" width
        self.smoothed = None                # L~_t
        self.prev = None                    # (state vector, n, action) of time step t - 1
        self.window, self.window_ms = [], 0.0
        self.bits = bits_min
        self.history = []                   # (m, bits) at every decision

    def _q_pair(self, x, n):
        out = self.net.q(x)
        keep = out[n - self.lo]
        more = out[n + 1 - self.lo] if n < self.hi else -np.inf
        return keep, more

    def _policy(self, x, n):
        keep, more = self._q_pair(x, n)
        greedy = 1 if more > keep else 0
        if n >= self.hi:
            return 0
        return 1 - greedy if self.rng.random() < self.eps else greedy

    def step(self, m, loss, elapsed_ms):
        """Global loss and wall time of training iteration m (0, 1, 2, ...); returns the width
        to use for iteration m.  Widths change only when m % T == 0 and never decrease."""
        self.window.append(float(loss))
        self.window_ms += float(elapsed_ms)
        if m % self.T != 0:
            return self.bits
        if self.smoothed is None:                                   # t = 0
            self.smoothed = np.full(self.T, float(loss))
            x = self.smoothed.copy()
            a = self._policy(x, self.n)
        else:
            losses = self.window[-self.T:]
            new_smoothed = smooth_losses(losses, self.smoothed[-1], self.alpha)
            x_prev, n_prev, a_prev = self.prev
            keep, more = self._q_pair(x_prev, n_prev)
            n_new = min(self.hi, n_prev + (1 if more > keep else 0))   # transition on the greedy action
            r = reward(new_smoothed, self.window_ms, self.scale)
            x = new_smoothed.copy()
            a = self._policy(x, n_new)
            q_new = self.net.q(x)[min(self.hi, n_new + a) - self.lo]
            idx_prev = min(self.hi, n_prev + a_prev) - self.lo
            delta = r + self.discount * q_new - self.net.q(x_prev)[idx_prev]
            self.net.td_step(x_prev, idx_prev, delta, self.lr)
            self.smoothed, self.n = new_smoothed, n_new
        self.prev = (x, self.n, a)
        self.bits = max(self.bits, min(self.hi, self.n + a))
        self.window, self.window_ms = [], 0.0
        self.history.append((m, self.bits))
        return self.bits


class WindowQSelector:
    """Every iteration: features = last `window` losses (relative to their mean), actions = the
    widths lo..hi, linear Q per action, one-step Q-learning, epsilon-greedy."""

    def __init__(self, window=10, bits_min=1, bits_max=8, epsilon=0.1, lr=0.05, discount=0.9,
                 reward_scale=300.0, seed=0):
        self.k, self.lo, self.hi = window, bits_min, bits_max
        self.eps, self.lr, self.discount, self.scale = epsilon, lr, discount, reward_scale
        self.rng = np.random.default_rng(seed)
        self.w = np.zeros((bits_max - bits_min + 1, window + 1))
        self.losses = []
        self.prev = None                    # (features, action index)

    def _features(self):
        v = np.array(([self.losses[0]] * self.k + self.losses)[-self.k:], np.float64)
        scale = max(abs(v).mean(), 1e-12)
        return np.concatenate([(v - v.mean()) / scale, [1.0]])

    def step(self, m, loss, elapsed_ms):
        self.losses.append(float(loss))
        x = self._features()
        q = self.w @ x
        if self.prev is not None:
            x_prev, a_prev = self.prev
            drop = self.losses[-2] - self.losses[-1]
            r = self.scale * drop / max(float(elapsed_ms), 1e-9)
            delta = r + self.discount * q.max() - self.w[a_prev] @ x_prev
            self.w[a_prev] += self.lr * delta * x_prev
        a = int(self.rng.integers(0, q.size)) if self.rng.random() < self.eps else int(np.argmax(q))
        self.prev = (x, a)
        return self.lo + a
