"""Pins for the oracle's sampling loop (Algorithm 1): the sequential sampler as a special case,
the drafter-equals-target run, losslessness on a toy Gaussian chain, round accounting."""
import numpy as np
from scipy import stats

import synth
from oracle import dit, drafter, schedule, trajectory


def _toy(N=12):
    sc = schedule.make("linear", N)
    A = np.array([[0.9, 0.2], [-0.1, 0.8]])

    def target(x, s):
        m = sc.coef_x[s] * x - sc.coef_eps[s] * (A @ x + 0.1 * s)
        return m, m.copy()
    return sc, A, target


def _sequential(x0, N, target, sigma2, noise):
    x = np.asarray(x0, np.float64)
    for n in range(1, N + 1):
        x = target(x, N - n)[0] + np.sqrt(sigma2[N - n]) * noise[n - 1]
    return x


def test_k0_is_the_sequential_sampler():
    N = 12
    sc, _, target = _toy(N)
    rng = np.random.default_rng(0)
    x0, zt = rng.standard_normal(2), rng.standard_normal((N, 2))
    x, st = trajectory.sample(x0, N, 0, target, None, sc.sigma2, zt, zt, rng.random(N))
    assert np.array_equal(x, _sequential(x0, N, target, sc.sigma2, zt))
    assert st["target_calls"] == N and st["parallel_efficiency"] == 1.0


def test_drafter_equal_to_target_accepts_everything():
    # Self-speculative run (Sec. 3.4): identical means give ell = 0, accepted for every u, so the
    # trajectory is the sequential one driven by the draft-role noise on drafted transitions.
    N, K = 14, 4
    sc, _, target = _toy(N)
    rng = np.random.default_rng(1)
    x0 = rng.standard_normal(2)
    zt, zd, u = rng.standard_normal((N, 2)), rng.standard_normal((N, 2)), np.ones(N)
    trace = []
    x, st = trajectory.sample(x0, N, K, target, lambda xp, f, s: target(xp, s), sc.sigma2, zt, zd, u, trace=trace)
    assert all(ok and ell == 0.0 for _, ok, ell in trace) and st["rejected"] == 0
    # rounds: a = 1, 6, 11 draft K = 4 transitions each (b <= N-1 = 13 caps the last to 12..13), then a = 14
    starts, a = [], 1
    noise = zd.copy()
    while a <= N:
        starts.append(a)
        noise[a - 1] = zt[a - 1]
        a = min(N - 1, a + K) + 1 if min(N - 1, a + K) > a else a + 1
    assert np.allclose(x, _sequential(x0, N, target, sc.sigma2, noise), atol=1e-13)
    n_draft_rounds = sum(min(N - 1, s + K) > s for s in starts)
    assert st["target_calls"] == len(starts) + n_draft_rounds
    assert st["parallel_efficiency"] == N / st["target_calls"] > 1.5


def test_lossless_on_a_gaussian_chain():
    # With a poor drafter the final state must still follow the sequential sampler's law
    # (Appendix B, unbiasedness applied transition by transition).
    N, K, n = 8, 3, 3000
    sc, A, target = _toy(N)

    def bad_draft(xp, f, s):
        m = target(xp, s)[0]
        return m + 0.6 * np.sqrt(sc.sigma2[s]) * np.array([1.0, -0.5]), f
    rng = np.random.default_rng(2)
    x0 = np.array([0.3, -0.2])
    spec, seq, rej = np.empty((n, 2)), np.empty((n, 2)), 0
    for i in range(n):
        zt, zd, u = rng.standard_normal((N, 2)), rng.standard_normal((N, 2)), rng.random(N)
        spec[i], st = trajectory.sample(x0, N, K, target, bad_draft, sc.sigma2, zt, zd, u)
        rej += st["rejected"]
        seq[i] = _sequential(x0, N, target, sc.sigma2, rng.standard_normal((N, 2)))
    assert rej > n // 2
    for c in range(2):
        assert stats.ks_2samp(spec[:, c], seq[:, c]).pvalue > 1e-3
    # planted mistake: accepting every draft without verification shifts the law and is caught
    biased = np.empty((n, 2))
    for i in range(n):
        zt, zd = rng.standard_normal((N, 2)), rng.standard_normal((N, 2))
        biased[i], _ = trajectory.sample(x0, N, K, target, bad_draft, sc.sigma2, zt, zd, np.zeros(N))
    assert min(stats.ks_2samp(biased[:, c], seq[:, c]).pvalue for c in range(2)) < 1e-6


def test_rejection_resumes_from_the_reflected_state():
    N, K = 10, 3
    sc, _, target = _toy(N)

    def off_draft(xp, f, s):
        return target(xp, s)[0] + 50.0 * np.sqrt(sc.sigma2[s]), f        # far off: always rejected
    rng = np.random.default_rng(3)
    x0, zt, zd = rng.standard_normal(2), rng.standard_normal((N, 2)), rng.standard_normal((N, 2))
    trace = []
    x, st = trajectory.sample(x0, N, K, target, off_draft, sc.sigma2, zt, zd, np.full(N, 0.5), trace=trace)
    assert st["accepted"] == 0 and all(not ok for _, ok, _ in trace)
    # every round finalises exactly two transitions (target step + reflected first draft) until the tail
    assert [t for t, _, _ in trace] == [2, 4, 6, 8]
    assert st["target_calls"] == 4 * 2 + 2 and st["accept_hist"][0] == 4


def test_tiny_dit_trajectory_runs_with_guidance_free_drafter():
    sh = synth.TINY
    N, K = 6, 3
    sc = schedule.make("linear", N)
    w = synth.make_target_weights(sh, 1, ada_std=0.2, out_gain=3.0)
    wd = synth.make_drafter_weights(sh, 2, ada_std=0.2, out_gain=3.0)
    label = 3

    def target(x, s):
        m, _, f = dit.verify_pass(w, sh, sc, x[None], [s], [label], 0.0)
        return m[0], f[0]

    def draft(xp, f, s):
        m, _, fn = drafter.guided_step(w, wd, sh, sc, xp, f, s, label, 0.0)
        return m, fn
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(4, 1, shape)
    zt, zd = synth.normal(4, 2, (N,) + shape), synth.normal(4, 3, (N,) + shape)
    u = synth.uniform01(4, 4, (N,))
    x, st = trajectory.sample(x0, N, K, target, draft, sc.sigma2, zt, zd, u)
    assert x.shape == shape and np.all(np.isfinite(x)) and st["draft_calls"] > 0
    assert st["accepted"] + st["rejected"] >= 1
