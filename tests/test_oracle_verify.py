"""Pins for the oracle's verifier: closed forms, the appendix's identities, Monte-Carlo laws."""
import numpy as np
import pytest
from scipy import stats

from oracle import verify as V

RNG = np.random.default_rng(1234)


def _case(d, s=0.3, sigma2=0.04):
    m = RNG.standard_normal(d)
    m_hat = m + s * RNG.standard_normal(d)
    x_hat = m_hat + np.sqrt(sigma2) * RNG.standard_normal(d)
    return m, m_hat, x_hat, sigma2


@pytest.mark.parametrize("d", [1, 3, 64, 1000])
def test_closed_form_equals_density_ratio(d):
    # Eq. qp: the closed form must equal the difference of the two Gaussian log-densities.
    m, m_hat, x_hat, s2 = _case(d)
    a = V.log_ratio(x_hat, m, m_hat, s2)
    b = V.log_ratio_definition(x_hat, m, m_hat, s2)
    assert abs(a - b) <= 1e-9 * max(1.0, abs(b))


def test_density_ratio_against_scipy():
    m, m_hat, x_hat, s2 = _case(5)
    ref = (stats.multivariate_normal(m, s2 * np.eye(5)).logpdf(x_hat)
           - stats.multivariate_normal(m_hat, s2 * np.eye(5)).logpdf(x_hat))
    assert abs(V.log_ratio(x_hat, m, m_hat, s2) - ref) < 1e-9 * max(1.0, abs(ref))


def test_reflection_1d_mirrors_about_midpoint():
    # Sec. 3.3: in one dimension x = 2 mid - x_hat.
    m, m_hat, x_hat = np.array([0.3]), np.array([-1.1]), np.array([0.7])
    assert np.allclose(V.reflect(x_hat, m, m_hat), m + m_hat - x_hat, atol=1e-15)


def test_reflection_identities():
    # Lemma 1 / Lemma 2: norm swaps, Re = -e, components orthogonal to e unchanged, involution.
    m, m_hat, x_hat, _ = _case(37)
    x = V.reflect(x_hat, m, m_hat)
    assert np.isclose(np.linalg.norm(x - m), np.linalg.norm(x_hat - m_hat), rtol=1e-13)
    assert np.isclose(np.linalg.norm(x - m_hat), np.linalg.norm(x_hat - m), rtol=1e-13)
    e = (m_hat - m) / np.linalg.norm(m_hat - m)
    r_in, r_out = x_hat - m_hat, x - m
    assert np.isclose(e @ r_out, -(e @ r_in), rtol=1e-12)
    assert np.allclose(r_out - e * (e @ r_out), r_in - e * (e @ r_in), atol=1e-13)
    # reflecting back with the roles of the two means swapped returns the draft
    assert np.allclose(V.reflect(x, m_hat, m), x_hat, atol=1e-12)
    # the mirror image of x_hat across the hyperplane through mid with normal e
    mid = 0.5 * (m + m_hat)
    assert np.allclose(x, x_hat - 2 * e * (e @ (x_hat - mid)), atol=1e-12)


def test_equal_means_always_accept_and_identity():
    m, _, _, s2 = _case(16)
    x_hat = m + 0.2 * RNG.standard_normal(16)
    for u in (0.0, 1e-30, 0.5, 1.0 - 1e-16, 1.0):
        x, ok, ell = V.verification(m, m, s2, x_hat, u)
        assert ok and ell == 0.0 and np.array_equal(x, x_hat)
    assert np.array_equal(V.reflect(x_hat, m, m), x_hat)


@pytest.mark.parametrize("delta_over_sigma", [0.25, 1.0, 2.5])
def test_acceptance_rate_matches_closed_form(delta_over_sigma):
    # Appendix D: E[a] = 2 Phi(-||m_p - m_q|| / (2 sigma)); rejection rate = total variation (Theorem 1).
    d, n, sigma = 6, 40000, 0.7
    rng = np.random.default_rng(7)
    m = rng.standard_normal(d)
    direction = rng.standard_normal(d)
    m_hat = m + delta_over_sigma * sigma * direction / np.linalg.norm(direction)
    acc = 0
    for _ in range(n):
        x_hat = m_hat + sigma * rng.standard_normal(d)
        acc += V.verification(m_hat, m, sigma ** 2, x_hat, rng.random())[1]
    expect = 2.0 * stats.norm.cdf(-delta_over_sigma / 2.0)
    se = np.sqrt(expect * (1 - expect) / n)
    assert abs(acc / n - expect) < 4.5 * se


def test_output_is_distributed_as_target():
    # Unbiasedness (Appendix B): the output is N(m, sigma^2 I) although the draft is N(m_hat, .).
    d, n, sigma = 4, 20000, 0.5
    rng = np.random.default_rng(11)
    m = rng.standard_normal(d)
    m_hat = m + np.array([0.6, -0.3, 0.1, 0.4])
    e = (m_hat - m) / np.linalg.norm(m_hat - m)
    out = np.empty((n, d))
    rejected = 0
    for i in range(n):
        x_hat = m_hat + sigma * rng.standard_normal(d)
        out[i], ok, _ = V.verification(m_hat, m, sigma ** 2, x_hat, rng.random())
        rejected += not ok
    assert rejected > n // 10          # the test exercises the reflection branch
    for c in range(d):
        assert stats.kstest((out[:, c] - m[c]) / sigma, "norm").pvalue > 1e-3
    assert stats.kstest(((out - m) @ e) / sigma, "norm").pvalue > 1e-3
    # a verifier that skipped the reflection (kept the mean-shifted draft) must fail this pin
    biased = m_hat + sigma * rng.standard_normal((n, d))
    assert stats.kstest(((biased - m) @ e) / sigma, "norm").pvalue < 1e-6


def test_relaxation_scale():
    m, m_hat, x_hat, s2 = _case(50, s=0.2)
    ell1 = V.log_ratio(x_hat, m, m_hat, s2, 1.0)
    assert V.log_ratio(x_hat, m, m_hat, s2) == ell1                       # lambda = 1 is the strict rule
    for lam in (0.5, 0.1, 0.0):
        assert np.isclose(V.log_ratio(x_hat, m, m_hat, s2, lam), lam * ell1, rtol=1e-12, atol=1e-300)
    # lambda -> 0 accepts everything; acceptance is monotone as lambda shrinks when ell < 0
    if ell1 < 0:
        u = np.exp(0.5 * ell1)        # rejected at lambda = 1
        oks = [V.verification(m_hat, m, s2, x_hat, u, lam)[1] for lam in (1.0, 0.75, 0.5, 0.25, 0.0)]
        assert oks[0] is False and oks[-1] is True
        assert all(b >= a for a, b in zip(oks, oks[1:]))
    # the reflection does not depend on lambda (e is a unit vector)
    xr1 = V.verification(m_hat, m, s2, x_hat, 1.0, 1.0)[0]
    xr2 = V.verification(m_hat, m, s2, x_hat, 1.0, 0.999)[0]
    if ell1 < 0:
        assert np.array_equal(xr1, xr2)


def _brute_first_reject(m, m_hat, x_hat, s2, u, lam, n_valid):
    B, K = u.shape
    n_acc = np.zeros(B, dtype=np.int32)
    for b in range(B):
        flags = []
        for k in range(n_valid[b]):
            ratio = np.exp(min(0.0, lam[b, k] * V.log_ratio_definition(x_hat[b, k], m[b, k], m_hat[b, k], s2[b, k])))
            flags.append(u[b, k] <= ratio)
        n_acc[b] = flags.index(False) if False in flags else len(flags)
    return n_acc


def test_first_reject_scan_against_brute_force():
    B, K, d = 40, 6, 24
    rng = np.random.default_rng(3)
    m = rng.standard_normal((B, K, d))
    m_hat = m + 0.15 * rng.standard_normal((B, K, d))
    s2 = rng.uniform(0.01, 0.1, (B, K))
    x_hat = m_hat + np.sqrt(s2)[..., None] * rng.standard_normal((B, K, d))
    u = rng.random((B, K))
    lam = rng.uniform(0.2, 1.0, (B, K))
    n_valid = rng.integers(0, K + 1, B)
    x_out, n_acc, ell = V.spec_verify(m, m_hat, x_hat, s2, u, lam, n_valid)
    assert np.array_equal(n_acc, _brute_first_reject(m, m_hat, x_hat, s2, u, lam, n_valid))
    assert 0 < n_acc.sum() < n_valid.sum()
    for b in range(B):
        j = n_acc[b]
        if n_valid[b] == 0:
            assert np.all(x_out[b] == 0)
        elif j == n_valid[b]:
            assert np.array_equal(x_out[b], x_hat[b, j - 1])
        else:
            assert np.allclose(x_out[b], V.reflect(x_hat[b, j], m[b, j], m_hat[b, j]))
            assert np.all(np.isnan(ell[b, j + 1:]))


def test_first_reject_extreme_uniforms():
    B, K, d = 5, 4, 8
    rng = np.random.default_rng(5)
    m = rng.standard_normal((B, K, d))
    m_hat = m + rng.standard_normal((B, K, d))
    s2 = np.full((B, K), 0.05)
    x_hat = m_hat + np.sqrt(0.05) * rng.standard_normal((B, K, d))
    _, n_acc, _ = V.spec_verify(m, m_hat, x_hat, s2, np.zeros((B, K)))
    assert np.all(n_acc == K)                                   # u = 0 accepts everything
    _, n_acc, ell = V.spec_verify(m, m_hat, x_hat, s2, np.ones((B, K)))
    for b in range(B):                                          # u = 1 accepts iff ell >= 0
        full = [V.log_ratio(x_hat[b, k], m[b, k], m_hat[b, k], 0.05) >= 0 for k in range(K)]
        assert n_acc[b] == (full.index(False) if False in full else K)


def test_sigma_must_be_positive():
    with pytest.raises(ValueError):
        V.verification(np.zeros(2), np.ones(2), 0.0, np.zeros(2), 0.5)


# ----------------------------------------------------------------------------- verification from the noise predictions
@pytest.mark.parametrize("G,shape", [(2, (4, 4, 6)), (1, (3, 5)), (2, (7,))])
def test_means_from_stream_eps_against_elementwise_loops(G, shape):
    rng = np.random.default_rng(G * 100 + len(shape))
    K, w_cfg = 3, 2.5
    eps = rng.standard_normal((K, G) + shape)
    x_first = rng.standard_normal(shape)
    x_hat = rng.standard_normal((K,) + shape)
    cx, ce = rng.uniform(1.0, 1.1, K), rng.uniform(0.01, 0.2, K)
    got = V.means_from_stream_eps(eps, x_first, x_hat, cx, ce, w_cfg)
    for k in range(K):
        x_k = x_first if k == 0 else x_hat[k - 1]
        for idx in np.ndindex(*shape):
            e = eps[(k, 0) + idx]
            if G == 2:
                e = eps[(k, 1) + idx] + w_cfg * (eps[(k, 0) + idx] - eps[(k, 1) + idx])
            assert abs(got[(k,) + idx] - (cx[k] * x_k[idx] - ce[k] * e)) < 1e-13


def test_means_from_stream_eps_special_cases():
    rng = np.random.default_rng(77)
    K, G, shape = 2, 2, (2, 4, 4)
    eps = rng.standard_normal((K, G) + shape)
    x_first, x_hat = rng.standard_normal(shape), rng.standard_normal((K,) + shape)
    one, zero = np.ones(K), np.zeros(K)
    # coef_eps = 0: the mean is the packed state itself -- x_first, then the drafts shifted by one slot
    m = V.means_from_stream_eps(eps, x_first, x_hat, one, zero, 3.0)
    assert np.array_equal(m[0], x_first) and np.array_equal(m[1], x_hat[0])
    # guidance scale 1 with two streams: the conditional stream alone; scale 0: the unconditional one
    m1 = V.means_from_stream_eps(eps, x_first, x_hat, zero, -one, 1.0)
    m0 = V.means_from_stream_eps(eps, x_first, x_hat, zero, -one, 0.0)
    assert np.allclose(m1, eps[:, 0], atol=1e-15) and np.allclose(m0, eps[:, 1], atol=1e-15)
    # one stream: the scale does not enter
    assert np.array_equal(V.means_from_stream_eps(eps[:, :1], x_first, x_hat, one, one, 3.0),
                          V.means_from_stream_eps(eps[:, :1], x_first, x_hat, one, one, 0.0))
    # equal to the schedule's own mean with guided eps (two independent routes to Eq. ddpm_update)
    from oracle import schedule as S
    sc = S.make("respaced", 50)
    idx = np.array([30, 29])
    m = V.means_from_stream_eps(eps, x_first, x_hat, sc.coef_x[idx], sc.coef_eps[idx], 4.0)
    for k in range(K):
        guided = eps[k, 1] + 4.0 * (eps[k, 0] - eps[k, 1])
        assert np.allclose(m[k], sc.mean(x_first if k == 0 else x_hat[k - 1], guided, int(idx[k])), atol=1e-14)


def test_spec_verify_from_eps_is_verification_of_those_means():
    rng = np.random.default_rng(5)
    B, K, G, shape = 3, 4, 2, (2, 4, 4)
    eps = 0.1 * rng.standard_normal((B, K, G) + shape)
    x_first = rng.standard_normal((B,) + shape)
    cx, ce = np.full((B, K), 1.01), np.full((B, K), 0.05)
    sigma2, u = np.full((B, K), 0.02), rng.uniform(0.0, 1.0, (B, K))
    # drafts built around the true means so that some are accepted and some are not
    x_hat = np.zeros((B, K) + shape); m_hat = np.zeros_like(x_hat)
    for b in range(B):
        for k in range(K):
            xk = x_first[b] if k == 0 else x_hat[b, k - 1]
            mk = V.means_from_stream_eps(eps[b, k:k + 1], xk, x_hat[b, :1], cx[b, k:k + 1], ce[b, k:k + 1], 2.0)[0]
            m_hat[b, k] = mk + 0.03 * rng.standard_normal(mk.shape)
            x_hat[b, k] = m_hat[b, k] + np.sqrt(sigma2[b, k]) * rng.standard_normal(mk.shape)
    x_out, n_acc, ell, means = V.spec_verify_from_eps(eps, x_first, m_hat, x_hat, cx, ce, 2.0, sigma2, u)
    assert 0 < n_acc.sum() < B * K            # a mix of outcomes
    for b in range(B):
        state = None
        for k in range(K):
            x, ok, l = V.verification(m_hat[b, k], means[b, k], sigma2[b, k], x_hat[b, k], u[b, k])
            assert abs(l - ell[b, k]) < 1e-12
            state = x
            if not ok:
                assert n_acc[b] == k
                break
        else:
            assert n_acc[b] == K
        assert np.allclose(x_out[b], state, atol=1e-15)
