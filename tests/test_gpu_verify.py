"""spec_verify (CUDA) against the oracle's Algorithm 2 on identical fp32 inputs."""
import numpy as np
import pytest
import torch

import synth
from oracle import schedule as osched
from oracle import verify as overify

pytestmark = pytest.mark.gpu

TOL_ELL = 1e-4          # decisions may differ only where |ell - log u| is below this (plus fp32 output rounding of ell)


def _run(m, mh, xh, s2, u, lam=None, n_valid=None):
    import paper_2511_20390_b200 as free
    cu = lambda a, dt=torch.float32: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    x, n, ell = free.spec_verify(cu(m), cu(mh), cu(xh), cu(s2), cu(u), lam=cu(lam),
                                 n_valid=cu(n_valid, torch.int32), want_logratio=True)
    torch.cuda.synchronize()
    return x.cpu().numpy(), n.cpu().numpy(), ell.cpu().numpy()


def _compare(m, mh, xh, s2, u, lam=None, n_valid=None):
    B, K = u.shape
    x, n, ell = _run(m, mh, xh, s2, u, lam, n_valid)
    xo, no, _ = overify.spec_verify(m, mh, xh, s2, u, lam, n_valid)
    nv = np.full(B, K) if n_valid is None else n_valid
    lam_ = np.ones((B, K)) if lam is None else lam
    n_exempt = 0
    for b in range(B):
        ell_o = np.array([overify.log_ratio(xh[b, k], m[b, k], mh[b, k], float(s2[b, k]), float(lam_[b, k]))
                          for k in range(nv[b])])
        if nv[b]:
            assert np.allclose(ell[b, :nv[b]], ell_o, rtol=2e-6, atol=1e-6)
        assert np.all(np.isnan(ell[b, nv[b]:]))
        if n[b] != no[b]:
            # allowed only if the deciding draft sits on the threshold
            k = min(n[b], no[b])
            assert abs(ell_o[k] - np.log(float(u[b, k]))) < TOL_ELL, (b, k, ell_o[k], u[b, k])
            n_exempt += 1
            continue
        if nv[b] == 0:
            assert np.all(x[b] == 0)
            continue
        scale = np.abs(xo[b]).max()
        assert np.abs(x[b] - xo[b]).max() <= 1e-5 * scale + 1e-7, b
    assert n_exempt <= max(1, B // 50)
    return n, no


@pytest.mark.parametrize("B,K,d,c", [(1, 6, 16384, 0.5), (3, 6, 16384, 1.0), (5, 16, 4096, 0.3), (2, 2, 16384, 50.0),
                                     (7, 8, 1000, 1.0), (4, 4, 1003, 0.7), (3, 64, 256, 0.2), (9, 3, 6, 1.5),
                                     (2, 5, 2048 + 4, 1.0), (33, 6, 16384, 0.8), (3, 6, 4096 + 1, 1.0),
                                     (100, 6, 16384, 0.8), (300, 2, 8192, 1.0), (4, 33, 16384, 0.5)])
def test_strict_matches_oracle(B, K, d, c):
    # c = |m_hat - m| / sigma of a typical draft: around 1 gives mixed decisions, 50 rejects at once
    sc = osched.make("respaced", 250)
    idx = np.linspace(5, 245, B * K).astype(int).reshape(B, K)
    s2 = sc.sigma2[idx].astype(np.float32)
    m, mh, xh, u = synth.verifier_inputs(100 + B + K, B, K, d, c * float(np.sqrt(s2.mean() / d)), s2)
    n, no = _compare(m, mh, xh, s2, u)
    assert n.min() >= 0 and n.max() <= K


def test_mixed_decisions_relaxed_and_ragged():
    B, K, d = 48, 6, 4096
    s2 = np.full((B, K), 0.02, np.float32)
    m, mh, xh, u = synth.verifier_inputs(7, B, K, d, 0.004, s2)       # |d|/sigma ~ 1.8: mixed accept / reject
    n, _ = _compare(m, mh, xh, s2, u)
    assert 0 < n.sum() < B * K and len(set(n.tolist())) >= 3
    lam = np.tile(synth.lambda_profile(K, floor=0.05, knee=0.5), (B, 1))
    n_rel, _ = _compare(m, mh, xh, s2, u, lam=lam)
    assert n_rel.sum() > n.sum() and np.all(n_rel >= n)                # relaxing never rejects earlier
    n1, _ = _compare(m, mh, xh, s2, u, lam=np.ones((B, K), np.float32))
    assert np.array_equal(n1, n)                                       # lambda = 1 is the strict rule
    nv = (np.arange(B) % (K + 1)).astype(np.int32)
    n_r, _ = _compare(m, mh, xh, s2, u, n_valid=nv)
    assert np.all(n_r <= nv)


@pytest.mark.parametrize("K", [2, 4, 6, 8, 16])
@pytest.mark.parametrize("s_rel", [0.01, 0.1, 1.0])
def test_sweep_strict_and_relaxed(K, s_rel):
    # the standalone sweep: d = 4x64x64, draft = target + N(0, s^2) with s relative to the step's sigma, per-step
    # variances from the 250-step schedule, strict rule and two relaxation levels
    B, d = 8, 16384
    sc = osched.make("respaced", 250)
    s2 = np.tile(sc.sigma2[np.linspace(240, 20, K).astype(int)].astype(np.float32), (B, 1))
    m, mh, xh, u = synth.verifier_inputs(300 + K, B, K, d, s_rel * float(np.sqrt(s2.mean())) / np.sqrt(d) * 8.0, s2)
    n_strict, _ = _compare(m, mh, xh, s2, u)
    prev = n_strict
    for lam_v in (0.5, 0.1):
        n_rel, _ = _compare(m, mh, xh, s2, u, lam=np.full((B, K), lam_v, np.float32))
        assert np.all(n_rel >= prev)                                   # a smaller lambda never rejects earlier
        prev = n_rel


def test_degenerate_cases():
    B, K, d = 4, 3, 512
    s2 = np.full((B, K), 0.05, np.float32)
    m, mh, xh, u = synth.verifier_inputs(9, B, K, d, 0.5, s2)
    # equal means: ell = 0, everything accepted even for u = 1
    x, n, ell = _run(m, m, xh, s2, np.ones((B, K), np.float32))
    assert np.all(n == K) and np.all(ell == 0) and np.array_equal(x, xh[:, -1])
    # u = 0 accepts everything
    x, n, _ = _run(m, mh, xh, s2, np.zeros((B, K), np.float32))
    assert np.all(n == K) and np.array_equal(x, xh[:, -1])
    # far-off drafts with u = 1: first draft rejected, reflection preserves the two norms (Lemma 2)
    x, n, _ = _run(m, mh, xh, s2, np.ones((B, K), np.float32))
    for b in range(B):
        if n[b] < K:
            j = n[b]
            assert np.isclose(np.linalg.norm(x[b] - m[b, j]), np.linalg.norm(xh[b, j] - mh[b, j]), rtol=1e-5)
            assert np.isclose(np.linalg.norm(x[b] - mh[b, j]), np.linalg.norm(xh[b, j] - m[b, j]), rtol=1e-5)
    # a non-positive variance is reported per sample and leaves x_out untouched
    bad = s2.copy(); bad[1, 0] = 0.0; bad[2, 2] = np.nan
    x, n, _ = _run(m, mh, xh, bad, u)
    assert n[1] == -5 and n[2] == -5 and n[0] >= 0 and n[3] >= 0 and np.all(x[1] == 0) and np.all(x[2] == 0)


def test_full_size_sweep_point_sampled_against_oracle():
    # largest point of the verifier sweep (K = 16, B = 256, d = 4x64x64): check a sample of the batch
    B, K, d = 256, 16, 16384
    sc = osched.make("respaced", 250)
    s2 = np.tile(sc.sigma2[np.linspace(240, 20, K).astype(int)].astype(np.float32), (B, 1))
    m, mh, xh, u = synth.verifier_inputs(21, B, K, d, 0.0015, s2)
    x, n, ell = _run(m, mh, xh, s2, u)
    pick = [0, 1, 77, 128, 200, 255]
    xo, no, _ = overify.spec_verify(m[pick], mh[pick], xh[pick], s2[pick], u[pick])
    assert np.array_equal(n[pick], no)
    assert np.abs(x[pick] - xo).max() <= 1e-5 * np.abs(xo).max()
    assert 0 < n.sum() < B * K
    # properties that hold for every sample: accepted prefix really passes, rejected draft really fails
    logu = np.log(u.astype(np.float64))
    for b in range(B):
        assert np.all(logu[b, :n[b]] <= np.minimum(0, ell[b, :n[b]]) + 1e-3)
        if n[b] < K:
            assert logu[b, n[b]] > min(0, ell[b, n[b]]) - 1e-3


def test_host_buffer_path():
    import paper_2511_20390_b200 as free
    B, K, d = 6, 6, 4096
    s2 = np.full((B, K), 0.03, np.float32)
    m, mh, xh, u = synth.verifier_inputs(5, B, K, d, 0.004, s2)
    x, n = free.spec_verify_host(m, mh, xh, s2, u)
    xo, no, _ = overify.spec_verify(m, mh, xh, s2, u)
    assert np.array_equal(n, no) and np.abs(x - xo).max() <= 1e-5 * np.abs(xo).max()
