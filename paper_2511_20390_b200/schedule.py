"""Host-side construction of the reverse-process tables passed to the library (`free_schedule`).

DDPM algebra of Eq. ddpm_update (Appendix "Variance Setting") with the fixed posterior variance of
Sec. 4 by default, other fixed-variance choices and the stochasticity family of Eq. mean_var_gamma as options,
evaluated in float64 on the host and stored as float32 device tables.  Schedule index
s = 0..N-1, s = N-1 the noisiest; transition n of a run uses s = N - n.
"""
import numpy as np


def _tables(betas, t_embed_value, variance="posterior", stochasticity=None):
    betas = np.asarray(betas, dtype=np.float64)
    alphas = 1.0 - betas
    abar = np.cumprod(alphas)
    abar_prev = np.append(1.0, abar[:-1])
    beta_tilde = (1.0 - abar_prev) / (1.0 - abar) * betas
    if stochasticity is not None:
        # Euler-Maruyama step of the epsilon-family of reverse processes (Appendix "Stochasticity Hyperparameter")
        k = 0.5 * (1.0 + float(stochasticity) ** 2)
        coef_x, coef_eps, sigma2 = 1.0 + betas / 2.0, k * betas / np.sqrt(1.0 - abar), float(stochasticity) ** 2 * betas
    else:
        coef_x, coef_eps = 1.0 / np.sqrt(alphas), betas / np.sqrt((1.0 - abar) * alphas)
        if variance == "posterior":
            sigma2 = beta_tilde
        elif variance == "beta":
            sigma2 = betas.copy()
        else:
            v = float(variance)
            if not 0.0 <= v <= 1.0:
                raise ValueError("variance must be 'posterior', 'beta' or a weight in [0, 1]")
            sigma2 = betas ** v * beta_tilde ** (1.0 - v)
    sigma2 = np.array(sigma2, dtype=np.float64)
    sigma2[0] = 0.0                       # the last transition adds no noise
    return {
        "coef_x": coef_x,
        "coef_eps": coef_eps,
        "sigma2": sigma2,
        "t_embed_value": np.asarray(t_embed_value, dtype=np.float64),
    }


def linear_schedule(N: int, beta_first: float = 1e-4, beta_last: float = 2e-2, variance="posterior", stochasticity=None) -> dict:
    """N-step schedule with beta linear between the two ends; the embedder sees s itself.
    variance: 'posterior' (Sec. 4), 'beta', or a log-domain interpolation weight in [0, 1] (Appendix "Variance
    Setting": any predefined sigma_t); stochasticity: the epsilon of Appendix "Stochasticity Hyperparameter"."""
    return _tables(np.linspace(beta_first, beta_last, N), np.arange(N), variance, stochasticity)


def respaced_schedule(N: int, N_full: int = 1000, beta_first: float = 1e-4, beta_last: float = 2e-2,
                      variance="posterior", stochasticity=None) -> dict:
    """N-step sub-schedule of an N_full-step linear one: abar kept at evenly spaced original indices,
    betas recomputed from consecutive abar ratios; the embedder sees the original index."""
    abar_full = np.cumprod(1.0 - np.linspace(beta_first, beta_last, N_full))
    keep = np.rint(np.arange(N) * ((N_full - 1) / (N - 1))).astype(np.int64)
    abar = abar_full[keep]
    betas = 1.0 - abar / np.append(1.0, abar[:-1])
    return _tables(betas, keep, variance, stochasticity)
