"""Reverse-process tables for `free_schedule`: argument marshalling around the library's host-side constructors.

The DDPM algebra itself (Eq. ddpm_update, the fixed posterior variance of Sec. 4, the other fixed-variance choices of
Appendix "Variance Setting" and the stochasticity family of Eq. mean_var_gamma) is computed in float64 by
`free_schedule_linear` / `free_schedule_respaced` of the C library.  Schedule index s = 0..N-1, s = N-1 the noisiest;
transition n of a run uses s = N - n.
"""
import ctypes as C

import numpy as np

_VAR_POSTERIOR, _VAR_BETA, _VAR_INTERP = 0, 1, 2


def _variance_args(variance):
    if variance == "posterior":
        return _VAR_POSTERIOR, 0.0
    if variance == "beta":
        return _VAR_BETA, 0.0
    v = float(variance)
    if not 0.0 <= v <= 1.0:
        raise ValueError("variance must be 'posterior', 'beta' or a weight in [0, 1]")
    return _VAR_INTERP, v


def _call(name, N, lead_args, variance, stochasticity):
    from .binding import lib, FreeError
    mode, weight = _variance_args(variance)
    out = {k: np.empty(N, dtype=np.float64) for k in ("coef_x", "coef_eps", "sigma2", "t_embed_value")}
    ptrs = [a.ctypes.data_as(C.c_void_p) for a in out.values()]
    rc = getattr(lib(), name)(*lead_args, mode, weight, -1.0 if stochasticity is None else float(stochasticity), *ptrs)
    if rc != 0:
        raise FreeError(rc, name)
    return out


def linear_schedule(N: int, beta_first: float = 1e-4, beta_last: float = 2e-2, variance="posterior", stochasticity=None) -> dict:
    """N-step schedule with beta linear between the two ends; the embedder sees s itself.
    variance: 'posterior' (Sec. 4), 'beta', or a log-domain interpolation weight in [0, 1] (Appendix "Variance
    Setting": any predefined sigma_t); stochasticity: the epsilon of Appendix "Stochasticity Hyperparameter".
    Returns float64 arrays coef_x, coef_eps, sigma2, t_embed_value of length N."""
    return _call("free_schedule_linear", N, (int(N), float(beta_first), float(beta_last)), variance, stochasticity)


def respaced_schedule(N: int, N_full: int = 1000, beta_first: float = 1e-4, beta_last: float = 2e-2,
                      variance="posterior", stochasticity=None) -> dict:
    """N-step sub-schedule of an N_full-step linear one: abar kept at evenly spaced original indices,
    betas recomputed from consecutive abar ratios; the embedder sees the original index."""
    return _call("free_schedule_respaced", N, (int(N), int(N_full), float(beta_first), float(beta_last)), variance, stochasticity)
