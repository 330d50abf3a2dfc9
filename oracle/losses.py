"""Drafter training objectives in fp64 (TEST INFRASTRUCTURE ONLY).

Sec. 3.2: noise MSE (Eq. mse), cosine feature loss (Eq. cos), Smooth-L1 on feature residuals
(Eqs. smooth, huber) and their weighted sum (Eq. free_loss).  Readings: the noise term is the mean
over elements (the text calls it a mean squared error; the equation prints the squared norm);
every term is averaged over the sequences of the batch; the small constant of Eq. cos is added to
the product of the two norms, as printed.
"""
import numpy as np


def noise_mse(eps_pred, eps_ref):
    """Eq. mse, as a mean over all elements."""
    d = np.asarray(eps_pred, np.float64) - np.asarray(eps_ref, np.float64)
    return float(np.mean(d * d))


def feature_cosine(f_pred, f_ref, eps_cos: float = 1e-8):
    """Eq. cos: mean over tokens of 1 - <p, r> / (|p| |r| + eps).  f: [..., N, D]."""
    p, r = np.asarray(f_pred, np.float64), np.asarray(f_ref, np.float64)
    dot = np.sum(p * r, axis=-1)
    den = np.sqrt(np.sum(p * p, axis=-1)) * np.sqrt(np.sum(r * r, axis=-1)) + eps_cos
    return float(np.mean(1.0 - dot / den))


def smooth_l1(f_pred, f_ref, beta: float = 1.0):
    """Eqs. smooth / huber: mean over tokens and channels of phi_beta(p - r),
    phi_beta(u) = u^2 / (2 beta) for |u| < beta, |u| - beta/2 otherwise."""
    u = np.abs(np.asarray(f_pred, np.float64) - np.asarray(f_ref, np.float64))
    return float(np.mean(np.where(u < beta, 0.5 * u * u / beta, u - 0.5 * beta)))


def free_loss(eps_pred, eps_ref, f_pred, f_ref, lambda_f: float, lambda_s: float, beta: float = 1.0,
              eps_cos: float = 1e-8):
    """Eq. free_loss.  Returns (L_noise, L_feat, L_smooth, L_total)."""
    ln = noise_mse(eps_pred, eps_ref)
    lf = feature_cosine(f_pred, f_ref, eps_cos)
    ls = smooth_l1(f_pred, f_ref, beta)
    return ln, lf, ls, ln + lambda_f * lf + lambda_s * ls
