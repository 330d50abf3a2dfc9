"""DDPM noise schedule, reverse-transition mean and fixed posterior variance.

Follows the one-step update of Appendix "Variance Setting" (Eq. ddpm_update):
    x_{t-1} = (x_t - (1 - alpha_t) / sqrt(1 - abar_t) * eps) / sqrt(alpha_t) + sigma_t z,
with sigma_t^2 fixed to the DDPM posterior variance beta~_t (Sec. 4).

Index convention: schedule index s = 0 .. N-1, s = N-1 being the noisiest.
The n-th transition of a sampling run (n = 1 .. N) uses s = N - n.
"""
import numpy as np


def linear_betas(N: int, beta_first: float = 1e-4, beta_last: float = 2e-2) -> np.ndarray:
    """beta_s linear in s from beta_first to beta_last (N values)."""
    return np.linspace(beta_first, beta_last, N, dtype=np.float64)


def respaced_betas(N: int, N_full: int = 1000, beta_first: float = 1e-4, beta_last: float = 2e-2):
    """Sub-sample an N_full-step linear schedule to N steps.

    Keeps abar at N evenly spaced original indices idx_i = round(i (N_full-1)/(N-1))
    and recomputes beta'_i = 1 - abar[idx_i] / abar[idx_{i-1}].  Returns (betas, idx);
    the timestep embedder is fed the original index idx_i.
    """
    abar_full = np.cumprod(1.0 - linear_betas(N_full, beta_first, beta_last))
    idx = np.rint(np.arange(N, dtype=np.float64) * (N_full - 1) / (N - 1)).astype(np.int64)
    abar = abar_full[idx]
    prev = np.concatenate([[1.0], abar[:-1]])
    return 1.0 - abar / prev, idx


class Schedule:
    """Per-index coefficient tables of the reverse transition.

    mean(x, eps, s) = coef_x[s] * x - coef_eps[s] * eps
    Default (Eq. ddpm_update, Sec. 4):
        coef_x = 1/sqrt(alpha_s), coef_eps = beta_s / (sqrt(1 - abar_s) sqrt(alpha_s)),
        sigma2[s] = beta~_s = beta_s (1 - abar_{s-1}) / (1 - abar_s),  abar_{-1} := 1.
    variance: other fixed-variance schedules (Appendix "Variance Setting" allows any predefined
        sigma_t): "beta" takes sigma2 = beta_s; a number v in [0, 1] interpolates the two in the log
        domain, sigma2 = beta_s^v beta~_s^(1-v).  The last transition (s = 0) keeps sigma = 0.
    stochasticity: the epsilon of Appendix "Stochasticity Hyperparameter" (Eq. mean_var_gamma): one
        Euler-Maruyama step of dY = (-f Y + (1+eps^2)/2 g^2 score) dt + eps g dW for the variance-
        preserving process whose step has gamma f = -beta_s/2, gamma g^2 = beta_s, with
        score = -eps_theta / sqrt(1 - abar_s):
        coef_x = 1 + beta_s/2, coef_eps = (1+eps^2)/2 beta_s / sqrt(1 - abar_s), sigma2 = eps^2 beta_s.
    """

    def __init__(self, betas: np.ndarray, t_embed_value=None, variance="posterior", stochasticity=None):
        betas = np.asarray(betas, dtype=np.float64)
        self.N = betas.shape[0]
        self.betas = betas
        self.alphas = 1.0 - betas
        self.abar = np.cumprod(self.alphas)
        abar_prev = np.concatenate([[1.0], self.abar[:-1]])
        posterior = betas * (1.0 - abar_prev) / (1.0 - self.abar)
        if stochasticity is None:
            self.coef_x = 1.0 / np.sqrt(self.alphas)
            self.coef_eps = betas / (np.sqrt(1.0 - self.abar) * np.sqrt(self.alphas))
            if variance == "posterior":
                self.sigma2 = posterior
            elif variance == "beta":
                self.sigma2 = betas.copy()
            else:
                v = float(variance)
                if not 0.0 <= v <= 1.0:
                    raise ValueError("variance interpolation weight must lie in [0, 1]")
                with np.errstate(divide="ignore", invalid="ignore"):
                    self.sigma2 = np.exp(v * np.log(betas) + (1.0 - v) * np.log(posterior))
            self.sigma2[0] = 0.0
        else:
            e2 = float(stochasticity) ** 2
            self.coef_x = 1.0 + 0.5 * betas
            self.coef_eps = 0.5 * (1.0 + e2) * betas / np.sqrt(1.0 - self.abar)
            self.sigma2 = e2 * betas
            self.sigma2[0] = 0.0
        self.t_embed_value = (np.arange(self.N, dtype=np.float64) if t_embed_value is None
                              else np.asarray(t_embed_value, dtype=np.float64))

    def mean(self, x, eps, s: int):
        return self.coef_x[s] * np.asarray(x, np.float64) - self.coef_eps[s] * np.asarray(eps, np.float64)


def make(kind: str, N: int, variance="posterior", stochasticity=None) -> Schedule:
    if kind == "linear":
        return Schedule(linear_betas(N), variance=variance, stochasticity=stochasticity)
    if kind == "respaced":
        b, idx = respaced_betas(N)
        return Schedule(b, t_embed_value=idx, variance=variance, stochasticity=stochasticity)
    raise ValueError(kind)
