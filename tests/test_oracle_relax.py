"""Pins for the relaxation-profile oracle (Sec. 3.4) and the library's host-side fit against it."""
import ctypes as C

import numpy as np
import pytest
from sklearn.isotonic import isotonic_regression

import synth
from oracle import relax


def test_isotonic_against_sklearn_and_brute_force():
    rng = np.random.default_rng(3)
    for n in (1, 2, 7, 40):
        y, w = rng.standard_normal(n).cumsum() * 0.3 + rng.standard_normal(n), rng.uniform(0.5, 3.0, n)
        g = relax.isotonic_increasing(y, w)
        assert np.allclose(g, isotonic_regression(y, sample_weight=w, increasing=True), atol=1e-12)
        assert np.all(np.diff(g) >= 0)
    # optimality on a tiny case: no other non-decreasing sequence on a grid does better
    y = np.array([1.0, 3.0, 2.0, 0.5])
    g = relax.isotonic_increasing(y)
    best = min(((np.array(c) - y) ** 2).sum() for c in np.ndindex(8, 8, 8, 8) if list(c) == sorted(c)
               for c in [np.array(c) * 0.5])
    assert ((g - y) ** 2).sum() <= best + 1e-12


def test_moving_average_keeps_order_and_constants():
    g = np.array([0.0, 0.0, 1.0, 1.0, 4.0, 9.0])
    for w in (0, 1, 2, 5):
        m = relax.moving_average(g, w)
        assert np.all(np.diff(m) >= -1e-15) and m[0] >= g[0] and m[-1] <= g[-1]
    assert np.array_equal(relax.moving_average(g, 0), g)
    assert np.allclose(relax.moving_average(np.full(5, 2.5), 2), 2.5)
    assert np.isclose(relax.moving_average(g, 1)[2], (0.0 + 1.0 + 1.0) / 3)


def test_lambda_profile_properties():
    N = 60
    g = np.linspace(0.5, 4.0, N) ** 2                       # already smooth and increasing
    lam = relax.lambda_profile(g)
    assert np.allclose(lam, g[0] / g, atol=1e-15)           # the fit leaves it alone: lambda = g_1 / g
    assert lam[0] == 1.0 and np.all(np.diff(lam) <= 0) and np.all(lam > 0) and np.all(lam <= 1)
    assert np.allclose(lam * g, g[0])                       # uniform scaled discrepancy
    assert np.allclose(relax.lambda_profile(7.3 * g), lam)  # the unit of the deviation does not matter
    assert np.array_equal(relax.lambda_profile(np.full(N, 0.2)), np.ones(N))
    assert np.array_equal(relax.lambda_profile(np.zeros(N)), np.ones(N))
    # a deviation curve built from a known table gives the table back
    true = synth.lambda_profile(N, floor=0.1, knee=0.5).astype(np.float64)
    assert np.allclose(relax.lambda_profile(0.03 / true), true / true[0], atol=1e-12)
    # noisy measurements: still monotone, in (0, 1], close to the clean answer after smoothing
    rng = np.random.default_rng(1)
    noisy = g * (1 + 0.05 * rng.standard_normal(N))
    ln = relax.lambda_profile(noisy, window=3)
    assert np.all(np.diff(ln) <= 1e-15) and ln[0] == 1.0 and np.abs(ln - lam).max() < 0.12


def test_unmeasured_transitions_take_the_nearest_value():
    e = np.array([0.0, 1.0, 0.0, 0.0, 2.0, 0.0])
    c = np.array([0, 4, 0, 0, 2, 0])
    lam = relax.lambda_profile(e, c)
    assert np.allclose(lam, [1, 1, 1, 0.5, 0.5, 0.5])       # gaps filled from the nearer side, the earlier one on a tie
    with pytest.raises(ValueError):
        relax.lambda_profile(e, np.zeros(6, int))


def test_recorder_identity_between_noise_and_mean_deviation():
    # |eps_pred - eps_ref| recorded from means equals the deviation of the noise predictions themselves
    from oracle import schedule
    sc = schedule.make("respaced", 50)
    rng = np.random.default_rng(2)
    x, e1, e2 = rng.standard_normal(30), rng.standard_normal(30), rng.standard_normal(30)
    rec = relax.Recorder(50, sc.coef_eps)
    t = 12
    rec(t, sc.mean(x, e1, 50 - t), sc.mean(x, e2, 50 - t), -0.3)
    dev, acc, cnt = rec.profile()
    assert np.isclose(dev[t - 1], np.linalg.norm(e1 - e2), rtol=1e-10) and np.isclose(acc[t - 1], np.exp(-0.3)) and cnt[t - 1] == 1
    assert cnt.sum() == 1


@pytest.mark.parametrize("seed,N,window,with_count", [(0, 50, 0, False), (1, 250, 4, True), (2, 7, 2, True), (3, 1, 1, False)])
def test_library_fit_matches_oracle(seed, N, window, with_count):
    from paper_2511_20390_b200 import binding
    rng = np.random.default_rng(seed)
    e = np.abs(np.linspace(0.2, 3.0, N) + 0.4 * rng.standard_normal(N))
    cnt = rng.integers(0, 5, N).astype(np.int64) if with_count else None
    if cnt is not None and cnt.sum() == 0:
        cnt[0] = 1
    lam = binding.fit_lambda_profile(e, cnt, window)
    ref = relax.lambda_profile(e, cnt, window)
    assert lam.dtype == np.float32 and np.allclose(lam, ref, rtol=1e-6, atol=1e-7)
    L = binding.lib()
    out = (C.c_float * N)()
    assert L.free_fit_lambda_profile(None, None, N, 0, out) != 0
    assert L.free_fit_lambda_profile(e.ctypes.data_as(C.c_void_p), None, N, -1, out) != 0
