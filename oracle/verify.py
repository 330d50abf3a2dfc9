"""Reflection-maximal-coupling verification in fp64 (TEST INFRASTRUCTURE ONLY).

Algorithm 2 ("Verification") for one draft, its relaxed acceptance (Eq. acc_relax)
and the sequential first-rejection loop of Algorithm 1.  Uniforms are arguments,
not drawn here, so every decision can be reproduced.
"""
import numpy as np


def log_ratio_definition(x_hat, m, m_hat, sigma2):
    """log N(x_hat; m, s2 I) - log N(x_hat; m_hat, s2 I), written out from the two
    Gaussian log-densities (Alg. 2, acceptance line)."""
    x_hat, m, m_hat = (np.asarray(a, np.float64).ravel() for a in (x_hat, m, m_hat))
    d = x_hat.size
    log_q = -0.5 * d * np.log(2.0 * np.pi * sigma2) - np.sum((x_hat - m) ** 2) / (2.0 * sigma2)
    log_p = -0.5 * d * np.log(2.0 * np.pi * sigma2) - np.sum((x_hat - m_hat) ** 2) / (2.0 * sigma2)
    return log_q - log_p


def log_ratio(x_hat, m, m_hat, sigma2, lam: float = 1.0):
    """Closed form of the log acceptance ratio (Eq. qp) with the relaxation scale (Eq. acc_relax):
    v = lam (m - m_hat);  ell = v^T (x_hat - mid) / sigma2,  mid = (m + m_hat)/2."""
    x_hat, m, m_hat = (np.asarray(a, np.float64).ravel() for a in (x_hat, m, m_hat))
    v = lam * (m - m_hat)
    mid = 0.5 * (m + m_hat)
    return float(v @ (x_hat - mid)) / sigma2


def reflect(x_hat, m, m_hat):
    """x = m + (I - 2 e e^T)(x_hat - m_hat),  e = (m_hat - m)/||m_hat - m||  (Alg. 2, else-branch).
    If the two means coincide the direction is undefined and the draft itself is returned."""
    x_hat, m, m_hat = (np.asarray(a, np.float64) for a in (x_hat, m, m_hat))
    diff = (m_hat - m).ravel()
    nrm = np.sqrt(diff @ diff)
    if nrm == 0.0:
        return x_hat.copy()
    e = diff / nrm
    r = (x_hat - m_hat).ravel()
    return (m.ravel() + r - 2.0 * e * (e @ r)).reshape(x_hat.shape)


def verification(m_hat, m, sigma2, x_hat, u, lam: float = 1.0):
    """Algorithm 2 for one draft.  Accept iff u <= min(1, exp(ell)), evaluated in the log domain
    (log u <= ell; u = 0 always accepts).  Returns (x, accepted, ell)."""
    if not sigma2 > 0.0:
        raise ValueError("sigma2 must be positive")
    ell = log_ratio(x_hat, m, m_hat, sigma2, lam)
    log_u = -np.inf if u <= 0.0 else np.log(u)
    if log_u <= min(0.0, ell):
        return np.asarray(x_hat, np.float64).copy(), True, ell
    return reflect(x_hat, m, m_hat), False, ell


def spec_verify(m, m_hat, x_hat, sigma2, u, lam=None, n_valid=None):
    """Sequential verification of K drafts per sample with a break at the first rejection
    (Alg. 1, verification loop).

    m, m_hat, x_hat: [B,K,...]; sigma2, u, lam: [B,K]; n_valid: [B] drafts present (default K).
    Returns x_out [B,...] (the last finalised state: the last accepted draft, or the reflection of
    the first rejected one), n_accept [B] (number of accepted drafts) and ell [B,K] (NaN where
    a draft was never examined).
    """
    m, m_hat, x_hat = (np.asarray(a, np.float64) for a in (m, m_hat, x_hat))
    B, K = m.shape[:2]
    sigma2 = np.broadcast_to(np.asarray(sigma2, np.float64), (B, K))
    u = np.broadcast_to(np.asarray(u, np.float64), (B, K))
    lam = np.ones((B, K)) if lam is None else np.broadcast_to(np.asarray(lam, np.float64), (B, K))
    n_valid = np.full(B, K, dtype=np.int64) if n_valid is None else np.asarray(n_valid, np.int64)
    x_out = np.zeros((B,) + m.shape[2:], dtype=np.float64)
    n_accept = np.zeros(B, dtype=np.int32)
    ell = np.full((B, K), np.nan)
    for b in range(B):
        for k in range(int(n_valid[b])):
            x, ok, ell[b, k] = verification(m_hat[b, k], m[b, k], sigma2[b, k], x_hat[b, k], u[b, k], lam[b, k])
            x_out[b] = x
            if not ok:
                break
            n_accept[b] += 1
    return x_out, n_accept, ell


def means_from_stream_eps(eps, x_first, x_hat, coef_x, coef_eps, cfg_scale):
    """Target means m_1..m_K of one sample from the noise predictions of its packed pass (Alg. 1,
    parallel-means line), so that verification can start from the network output itself.

    eps [K, G, ...]: per packed state the prediction of G = 2 streams (conditional, then
    unconditional) under guidance, else of one.  Packed state k is x_first for k = 0 and the draft
    x_hat[k-1] after that (the pass sees the current state and the first K-1 drafts).
    eps_k = eps_u + w (eps_c - eps_u) with w = cfg_scale (the single stream when G = 1);
    m_k = coef_x[k] x_k - coef_eps[k] eps_k  (Eq. ddpm_update).  Returns [K, ...]."""
    eps = np.asarray(eps, np.float64)
    K, G = eps.shape[:2]
    x_hat = np.asarray(x_hat, np.float64)
    means = np.zeros_like(x_hat)
    for k in range(K):
        e = eps[k, 0] if G == 1 else eps[k, 1] + cfg_scale * (eps[k, 0] - eps[k, 1])
        x_k = np.asarray(x_first, np.float64) if k == 0 else x_hat[k - 1]
        means[k] = coef_x[k] * x_k - coef_eps[k] * e
    return means


def spec_verify_from_eps(eps, x_first, m_hat, x_hat, coef_x, coef_eps, cfg_scale, sigma2, u, lam=None, n_valid=None):
    """means_from_stream_eps for every sample, then the sequential verification loop.
    eps [B,K,G,...]; x_first [B,...]; m_hat, x_hat [B,K,...]; coef_x, coef_eps, sigma2, u, lam [B,K].
    Returns (x_out, n_accept, ell, means)."""
    B = len(eps)
    means = np.stack([means_from_stream_eps(eps[b], x_first[b], x_hat[b], coef_x[b], coef_eps[b], cfg_scale)
                      for b in range(B)])
    x_out, n_accept, ell = spec_verify(means, m_hat, x_hat, sigma2, u, lam, n_valid)
    return x_out, n_accept, ell, means
