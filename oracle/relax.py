"""Uncertainty-guided relaxation profile in fp64 (TEST INFRASTRUCTURE ONLY).

Sec. 3.4: an offline speculative run records, per denoising step, the deviation between the
drafter's and the target's noise predictions and the acceptance probability; a smooth,
monotonically increasing curve is fitted to the deviations, inverted and rescaled to [0, 1].
Readings taken where the paper names no procedure: the monotone fit is the least-squares
non-decreasing sequence (isotonic regression), smoothing is a centred moving average with the
ends held, and "inverse rescaled to [0, 1]" is lambda_n = g_1 / g_n (1 at the first transition,
lambda_n g_n constant); steps without a measurement take the nearest measured value.
"""
import numpy as np


class Recorder:
    """Collects, per transition n = 1..N, what the verifier saw for every examined draft.  Both means
    of a draft are computed from the same packed state x, m = coef_x x - coef_eps eps
    (Eq. ddpm_update), hence eps_pred - eps_ref = (m - m_hat) / coef_eps."""

    def __init__(self, N, coef_eps):
        self.N, self.coef_eps = N, np.asarray(coef_eps, np.float64)
        self.dev = np.zeros(N); self.acc = np.zeros(N); self.count = np.zeros(N, np.int64)

    def __call__(self, t, m_hat, m, ell):
        s = self.N - t                                        # schedule index of transition t
        diff = (np.asarray(m, np.float64) - np.asarray(m_hat, np.float64)).ravel() / self.coef_eps[s]
        self.dev[t - 1] += np.sqrt(diff @ diff)
        self.acc[t - 1] += min(1.0, np.exp(ell))
        self.count[t - 1] += 1

    def profile(self):
        c = np.maximum(self.count, 1)
        return self.dev / c, self.acc / c, self.count.copy()


def isotonic_increasing(y, w=None):
    """argmin_g sum w_i (g_i - y_i)^2 subject to g_1 <= g_2 <= ... : merge neighbouring blocks that
    violate the order into their weighted mean until none is left."""
    y = np.asarray(y, np.float64)
    w = np.ones_like(y) if w is None else np.asarray(w, np.float64)
    blocks = [[y[i], w[i], 1] for i in range(len(y))]
    i = 0
    while i + 1 < len(blocks):
        if blocks[i][0] > blocks[i + 1][0]:
            a, b = blocks[i], blocks[i + 1]
            blocks[i:i + 2] = [[(a[0] * a[1] + b[0] * b[1]) / (a[1] + b[1]), a[1] + b[1], a[2] + b[2]]]
            i = max(i - 1, 0)
        else:
            i += 1
    return np.concatenate([np.full(n, v) for v, _, n in blocks])


def moving_average(g, window):
    """Centred mean over 2*window+1 points, indices clamped to the ends."""
    g = np.asarray(g, np.float64)
    idx = np.clip(np.arange(len(g))[:, None] + np.arange(-window, window + 1)[None, :], 0, len(g) - 1)
    return g[idx].mean(axis=1)


def lambda_profile(eps_delta, count=None, window=0):
    """lambda[n-1], n = 1..N, from the measured deviations (Sec. 3.4)."""
    e = np.asarray(eps_delta, np.float64)
    N = len(e)
    ok = np.isfinite(e) & (e >= 0) & (np.ones(N, bool) if count is None else np.asarray(count) > 0)
    valid = np.flatnonzero(ok)
    if len(valid) == 0:
        raise ValueError("no measured transition")
    nearest = np.array([valid[np.argmin(np.abs(valid - n))] for n in range(N)])     # argmin takes the earlier one on a tie
    y = e[nearest]
    w = np.ones(N) if count is None else np.where(ok, np.asarray(count, np.float64), 1.0)
    g = moving_average(isotonic_increasing(y, w), window)
    with np.errstate(divide="ignore", invalid="ignore"):
        lam = np.where(g > 0, np.minimum(g[0] / g, 1.0), 1.0)
    return lam
