"""Host-side construction of the reverse-process tables passed to the library (`free_schedule`).

DDPM algebra of Eq. ddpm_update (Appendix "Variance Setting") with the fixed posterior variance of
Sec. 4, evaluated in float64 on the host and stored as float32 device tables.  Schedule index
s = 0..N-1, s = N-1 the noisiest; transition n of a run uses s = N - n.
"""
import numpy as np


def _tables(betas, t_embed_value):
    betas = np.asarray(betas, dtype=np.float64)
    alphas = 1.0 - betas
    abar = np.cumprod(alphas)
    abar_prev = np.append(1.0, abar[:-1])
    return {
        "coef_x": 1.0 / np.sqrt(alphas),
        "coef_eps": betas / np.sqrt((1.0 - abar) * alphas),
        "sigma2": (1.0 - abar_prev) / (1.0 - abar) * betas,
        "t_embed_value": np.asarray(t_embed_value, dtype=np.float64),
    }


def linear_schedule(N: int, beta_first: float = 1e-4, beta_last: float = 2e-2) -> dict:
    """N-step schedule with beta linear between the two ends; the embedder sees s itself."""
    return _tables(np.linspace(beta_first, beta_last, N), np.arange(N))


def respaced_schedule(N: int, N_full: int = 1000, beta_first: float = 1e-4, beta_last: float = 2e-2) -> dict:
    """N-step sub-schedule of an N_full-step linear one: abar kept at evenly spaced original indices,
    betas recomputed from consecutive abar ratios; the embedder sees the original index."""
    abar_full = np.cumprod(1.0 - np.linspace(beta_first, beta_last, N_full))
    keep = np.rint(np.arange(N) * ((N_full - 1) / (N - 1))).astype(np.int64)
    abar = abar_full[keep]
    betas = 1.0 - abar / np.append(1.0, abar[:-1])
    return _tables(betas, keep)
