"""Seeded synthetic workloads: verifier operands, packed-state batches, relaxation tables.

These stand in for the paper's ImageNet 256^2 / 512^2 latents (Sec. 4): only the
shapes and value ranges are taken from there (4x32x32 / 4x64x64 latents with
unit-variance entries, class ids 0..999).
"""
import numpy as np

from .rng import normal, uniform01, _gen


def verifier_inputs(seed: int, B: int, K: int, d: int, s: float, sigma2: np.ndarray):
    """Operands of the acceptance test for B samples x K drafts of dimension d.

    Target means are N(0,1); each draft mean is the target mean plus N(0, s^2)
    noise; each draft sample is its draft mean plus sqrt(sigma2[b,k]) * N(0,1);
    uniforms are in (0,1).  `sigma2` is [B,K] (or broadcastable to it).
    Returns fp32 arrays m, m_hat, x_hat of shape [B,K,d] and u of shape [B,K].
    """
    sigma2 = np.broadcast_to(np.asarray(sigma2, dtype=np.float64), (B, K))
    m = normal(seed, 11, (B, K, d))
    m_hat = (m + np.float32(s) * normal(seed, 12, (B, K, d))).astype(np.float32)
    z = normal(seed, 13, (B, K, d))
    x_hat = (m_hat + np.sqrt(sigma2).astype(np.float32)[..., None] * z).astype(np.float32)
    u = uniform01(seed, 14, (B, K))
    return m, m_hat, x_hat, u


def lambda_profile(N: int, floor: float = 0.1, knee: float = 0.6, width: float = 0.12) -> np.ndarray:
    """Synthetic relaxation table lambda[n], n = 0..N-1 in sampling order (n = 0 is
    the first, noisiest transition).

    The paper obtains its table from a curve fitted to measurements on a trained
    model, which are not available; this stand-in has the stated properties only:
    values in (0, 1], equal to 1 at the start, non-increasing ("strict to loose").
    """
    n = np.arange(N, dtype=np.float64) / max(N - 1, 1)
    g = 1.0 + (1.0 / floor - 1.0) / (1.0 + np.exp(-(n - knee) / width))   # increasing "uncertainty" curve
    lam = g[0] / g
    return lam.astype(np.float32)


def pack_states(seed: int, B: int, K: int, d_shape, n_sched: int, n_classes: int):
    """A batch of packed verification inputs.

    For each of B samples: K latent states (the current state followed by K-1
    drafted states) at K consecutive transitions, i.e. K distinct schedule
    indices descending by one, starting at a random point of the schedule, and
    one class label shared by the K states.
    Returns x [B,K,*d_shape] fp32, t_idx [B,K] int32, labels [B,K] int32.
    """
    g = _gen(seed, 31)
    x = normal(seed, 32, (B, K) + tuple(d_shape))
    hi = g.integers(low=K, high=n_sched, size=B)          # schedule index of the first packed state
    t_idx = (hi[:, None] - 1 - np.arange(K)[None, :]).astype(np.int32)
    labels = np.repeat(g.integers(low=0, high=n_classes, size=(B, 1)), K, axis=1).astype(np.int32)
    return x, t_idx, labels


def eps_verifier_inputs(seed: int, B: int, K: int, G: int, d_shape, s: float, sigma2: np.ndarray, eps_std: float = 1.0):
    """Operands of a verification that starts from a network's noise predictions.

    eps [B,K,G,*d_shape] is N(0, eps_std^2).  The state chain is x_first ~ N(0,1) followed by the
    drafts themselves: each draft mean is its predecessor in the chain plus N(0, s^2) noise, each
    draft sample its draft mean plus sqrt(sigma2[b,k]) * N(0,1); uniforms are in (0,1).
    Returns fp32 arrays eps, x_first [B,*d_shape], m_hat, x_hat [B,K,*d_shape] and u [B,K].
    """
    sigma2 = np.broadcast_to(np.asarray(sigma2, dtype=np.float64), (B, K))
    d_shape = tuple(d_shape)
    eps = normal(seed, 41, (B, K, G) + d_shape, std=eps_std)
    x_first = normal(seed, 42, (B,) + d_shape)
    n = normal(seed, 43, (B, K) + d_shape)
    z = normal(seed, 44, (B, K) + d_shape)
    m_hat = np.zeros((B, K) + d_shape, np.float32)
    x_hat = np.zeros((B, K) + d_shape, np.float32)
    prev = x_first
    for k in range(K):
        m_hat[:, k] = prev + np.float32(s) * n[:, k]
        x_hat[:, k] = m_hat[:, k] + np.sqrt(sigma2[:, k]).astype(np.float32).reshape((B,) + (1,) * len(d_shape)) * z[:, k]
        prev = x_hat[:, k]
    u = uniform01(seed, 45, (B, K))
    return eps, x_first, m_hat, x_hat, u
