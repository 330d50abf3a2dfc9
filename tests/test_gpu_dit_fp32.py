"""fp32 mode (CUDA cores) against the fp64 oracle: single kernels, the packed pass, the drafter step and
the whole sampling loop on the tiny configuration.  Tolerance 1e-4 (max error / max |oracle|)."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit as odit, drafter as odrafter, schedule as osched, trajectory as otraj
from gpu_util import cu, nerr

pytestmark = pytest.mark.gpu
TOL = 1e-4


@pytest.fixture(scope="module")
def free():
    import paper_2511_20390_b200 as f
    f.lib()
    return f


@pytest.mark.parametrize("M,N,K", [(96, 192, 64), (7, 5, 3), (130, 65, 33), (64, 64, 16), (1, 300, 257)])
def test_linear_epilogues(free, M, N, K):
    from paper_2511_20390_b200 import binding as b
    rng = np.random.default_rng(M + N + K)
    A, W, bias = rng.standard_normal((M, K)), rng.standard_normal((N, K)) * 0.2, rng.standard_normal(N)
    ref = odit.linear(A, W, bias)
    assert nerr(b.op_linear(cu(A), cu(W), cu(bias)), ref) < TOL
    assert nerr(b.op_linear(cu(A), cu(W), cu(bias), epilogue=b.EPI_BIAS_GELU), odit.gelu_tanh(ref)) < TOL
    assert nerr(b.op_linear(cu(A), cu(W), cu(bias), epilogue=b.EPI_BIAS_SILU), odit.silu(ref)) < TOL
    rps = 4
    nseq = (M + rps - 1) // rps
    gate, resid = rng.standard_normal((nseq, 3 * N)), rng.standard_normal((M, N))
    g = cu(gate)[:, N:2 * N]                       # a strided view: gate rows sit inside a wider table
    out = b.op_linear(cu(A), cu(W), cu(bias), epilogue=b.EPI_GATE_RESIDUAL, resid=cu(resid), gate=g, rows_per_seq=rps)
    ref_r = resid + np.repeat(gate[:, N:2 * N], rps, axis=0)[:M] * ref
    assert nerr(out, ref_r) < TOL


@pytest.mark.parametrize("M,D,rps", [(32, 64, 16), (20, 384, 5), (9, 1152, 3), (5, 100, 2)])
def test_ln_modulate(free, M, D, rps):
    from paper_2511_20390_b200 import binding as b
    rng = np.random.default_rng(D)
    x = rng.standard_normal((M, D)) * 3 + 1
    nseq = (M + rps - 1) // rps
    mod = rng.standard_normal((nseq, 6 * D)) * 0.5
    ref = odit.layer_norm(x) * (1 + np.repeat(mod[:, D:2 * D], rps, 0)[:M]) + np.repeat(mod[:, :D], rps, 0)[:M]
    m = cu(mod)
    assert nerr(b.op_ln_modulate(cu(x), m[:, :D], m[:, D:2 * D], rps), ref) < TOL
    assert nerr(b.op_ln_modulate(cu(x), m[:, :D], m[:, D:2 * D], rps, out_dtype=b.FREE_BF16), ref) < 8e-3


@pytest.mark.parametrize("n_seq,T,h,dh", [(2, 16, 2, 32), (1, 50, 3, 24), (3, 256, 2, 64), (1, 33, 1, 72)])
def test_attention(free, n_seq, T, h, dh):
    from paper_2511_20390_b200 import binding as b
    rng = np.random.default_rng(T)
    qkv = rng.standard_normal((n_seq, T, 3, h, dh))
    ref = np.empty((n_seq, T, h * dh))
    for s in range(n_seq):
        for a in range(h):
            ref[s, :, a * dh:(a + 1) * dh] = odit.attention(qkv[s, :, 0, a], qkv[s, :, 1, a], qkv[s, :, 2, a])
    got = b.op_attention(cu(qkv.reshape(n_seq, T, 3 * h * dh)), h)
    assert nerr(got, ref) < TOL


def _tiny_model(free, cfg_gain=1.0, with_drafter=True):
    sh = synth.TINY
    w = synth.make_target_weights(sh, 1, ada_std=0.2, out_gain=cfg_gain)
    wd = synth.make_drafter_weights(sh, 2, ada_std=0.2, out_gain=cfg_gain)
    model = free.Model(sh, w, wd if with_drafter else None, dtype="fp32")
    return sh, w, wd, model


@pytest.mark.parametrize("cfg", [0.0, 4.0])
def test_packed_pass_tiny(free, cfg):
    sh, w, wd, model = _tiny_model(free)
    sc = osched.make("linear", 50)
    dsched = free.DeviceSchedule(free.linear_schedule(50))
    x, t, y = synth.pack_states(3, 1, 6, (sh.C, sh.H, sh.W), 50, sh.n_classes)
    x, t, y = x[0], t[0], y[0]
    mean, eps, feat = model.dit_verify_pass(cu(x), cu(t, torch.int32), cu(y, torch.int32), cfg, dsched, want_eps=True, want_feat=True)
    torch.cuda.synchronize()
    mo, eo, fo = odit.verify_pass(w, sh, sc, x, t, y, cfg)
    assert nerr(eps, eo) < TOL and nerr(mean, mo) < TOL and nerr(feat, fo) < TOL
    assert feat.shape[1] == (2 if cfg else 1)


def test_packed_pass_is_batch_invariant(free):
    sh, w, wd, model = _tiny_model(free)
    dsched = free.DeviceSchedule(free.linear_schedule(50))
    x, t, y = synth.pack_states(5, 3, 6, (sh.C, sh.H, sh.W), 50, sh.n_classes)
    X, T, Y = cu(x.reshape(18, *x.shape[2:])), cu(t.reshape(-1), torch.int32), cu(y.reshape(-1), torch.int32)
    all_ = model.dit_verify_pass(X, T, Y, 4.0, dsched).clone()
    one = model.dit_verify_pass(X[7:8].contiguous(), T[7:8].contiguous(), Y[7:8].contiguous(), 4.0, dsched)
    assert torch.equal(all_[7:8], one)


@pytest.mark.parametrize("cfg", [0.0, 4.0])
def test_draft_step_tiny(free, cfg):
    sh, w, wd, model = _tiny_model(free)
    sc = osched.make("linear", 50)
    dsched = free.DeviceSchedule(free.linear_schedule(50))
    n, G = 3, (2 if cfg else 1)
    x = synth.normal(8, 1, (n, sh.C, sh.H, sh.W))
    f = synth.normal(8, 2, (n, G, sh.n_tok, sh.D))
    z = synth.normal(8, 3, (n, sh.C, sh.H, sh.W))
    t, y = np.array([40, 12, 3], np.int32), np.array([1, 9, 4], np.int32)
    m_hat, x_hat, f_next = model.draft_step(cu(x), cu(f), cu(t, torch.int32), cu(y, torch.int32), cfg, dsched, cu(z))
    torch.cuda.synchronize()
    for i in range(n):
        mo, eo, fo = odrafter.guided_step(w, wd, sh, sc, x[i], f[i], int(t[i]), int(y[i]), cfg)
        assert nerr(m_hat[i], mo) < TOL and nerr(f_next[i], fo) < TOL
        assert nerr(x_hat[i], mo + np.sqrt(sc.sigma2[t[i]]) * z[i]) < TOL


def _oracle_traj(sh, w, wd, sc, N, K, cfg, x0, label, zt, zd, u, lam=None):
    def target(x, s):
        m, _, f = odit.verify_pass(w, sh, sc, x[None], [s], [label], cfg)
        return m[0], f[0]

    def draft(xp, f, s):
        m, _, fn = odrafter.guided_step(w, wd, sh, sc, xp, f, s, label, cfg)
        return m, fn
    trace = []
    x, st = otraj.sample(x0, N, K, target, draft, sc.sigma2, zt, zd, u, lam=lam, trace=trace)
    return x, st, trace


@pytest.mark.parametrize("K,cfg,relaxed", [(6, 0.0, False), (0, 0.0, False), (3, 4.0, True)])
def test_trajectory_tiny_matches_oracle(free, K, cfg, relaxed):
    sh, w, wd, model = _tiny_model(free)
    N, B = 50, 2
    sc = osched.make("linear", N)
    dsched = free.DeviceSchedule(free.linear_schedule(N))
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(4, 1, (B,) + shape)
    zt, zd = synth.normal(4, 2, (B, N) + shape), synth.normal(4, 3, (B, N) + shape)
    u = synth.uniform01(4, 4, (B, N))
    labels = np.array([3, 7], np.int32)
    lam = synth.lambda_profile(N, floor=0.2) if relaxed else None
    xf, st = model.sample_trajectory(cu(x0), cu(labels, torch.int32), dsched, K, cfg, cu(zt), cu(zd), cu(u),
                                     lam=cu(lam) if relaxed else None)
    acc = rej = calls = 0
    for b in range(B):
        xo, so, trace = _oracle_traj(sh, w, wd, sc, N, K, cfg, x0[b], int(labels[b]), zt[b], zd[b], u[b], lam)
        # decisions are only comparable away from the threshold
        assert all(abs(ell - np.log(u[b, t - 1])) > 1e-3 for t, ok, ell in trace if ell < 0)
        assert nerr(xf[b], xo) < 5 * TOL
        acc += so["accepted"]; rej += so["rejected"]; calls += so["target_calls"]
    assert st["accepted"] == acc and st["rejected"] == rej and st["target_calls"] == calls
    assert abs(st["parallel_efficiency"] - B * N / calls) < 1e-12
    if K == 6:
        assert acc > 5 and rej > 5
    if K == 0:
        assert st["target_calls"] == B * N and st["draft_calls"] == 0


@pytest.mark.parametrize("K,cfg", [(4, 0.0), (3, 4.0)])
def test_uncertainty_profile_tiny_matches_oracle(free, K, cfg):
    """The offline run of Sec. 3.4 (per-transition prediction deviation and acceptance probability of every examined
    draft) against the oracle's recorder on the same trajectories, and the relaxation table fitted from it."""
    from oracle import relax as orelax
    sh, w, wd, model = _tiny_model(free)
    N, B = 50, 2
    sc = osched.make("linear", N)
    dsched = free.DeviceSchedule(free.linear_schedule(N))
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(6, 1, (B,) + shape)
    zt, zd = synth.normal(6, 2, (B, N) + shape), synth.normal(6, 3, (B, N) + shape)
    u = synth.uniform01(6, 4, (B, N))
    labels = np.array([2, 8], np.int32)
    dev, acc, cnt = model.uncertainty_profile(cu(x0), cu(labels, torch.int32), dsched, K, cfg, cu(zt), cu(zd), cu(u))
    rec = orelax.Recorder(N, sc.coef_eps)
    for b in range(B):
        def target(x, s, b=b):
            m, _, f = odit.verify_pass(w, sh, sc, x[None], [s], [int(labels[b])], cfg)
            return m[0], f[0]

        def draft(xp, f, s, b=b):
            m, _, fn = odrafter.guided_step(w, wd, sh, sc, xp, f, s, int(labels[b]), cfg)
            return m, fn
        trace = []
        otraj.sample(x0[b], N, K, target, draft, sc.sigma2, zt[b], zd[b], u[b], trace=trace, observe=rec)
        assert all(abs(ell - np.log(u[b, t - 1])) > 1e-3 for t, ok, ell in trace if ell < 0)
    dev_o, acc_o, cnt_o = rec.profile()
    assert np.array_equal(cnt, cnt_o) and cnt.sum() > 10 and cnt[0] == 0 and cnt[-1] == 0
    seen = cnt > 0
    assert np.allclose(dev[seen], dev_o[seen], rtol=1e-3) and np.all(dev[~seen] == 0)
    assert np.allclose(acc[seen], acc_o[seen], atol=2e-3)
    lam = free.fit_lambda_profile(dev, cnt, 2)
    assert np.allclose(lam, orelax.lambda_profile(dev_o, cnt_o, 2), rtol=2e-3)
    assert lam[0] == 1.0 and np.all(np.diff(lam) <= 0) and np.all(lam > 0)


@pytest.mark.parametrize("kw", [{"stochasticity": 0.7}, {"variance": "beta"}, {"variance": 0.5}])
def test_trajectory_with_other_variance_schedules(free, kw):
    """Other fixed-variance schedules and the stochasticity family (Appendices "Variance Setting" / "Stochasticity
    Hyperparameter") are tables to the kernels: the whole loop against the oracle with the oracle's own tables."""
    sh, w, wd, model = _tiny_model(free)
    N, B, K, cfg = 50, 2, 4, 0.0
    sc = osched.make("linear", N, **kw)
    dsched = free.DeviceSchedule(free.linear_schedule(N, **kw))
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(14, 1, (B,) + shape)
    zt, zd = synth.normal(14, 2, (B, N) + shape), synth.normal(14, 3, (B, N) + shape)
    u = synth.uniform01(14, 4, (B, N))
    labels = np.array([1, 6], np.int32)
    xf, st = model.sample_trajectory(cu(x0), cu(labels, torch.int32), dsched, K, cfg, cu(zt), cu(zd), cu(u))
    acc = rej = 0
    for b in range(B):
        xo, so, trace = _oracle_traj(sh, w, wd, sc, N, K, cfg, x0[b], int(labels[b]), zt[b], zd[b], u[b])
        assert all(abs(ell - np.log(u[b, t - 1])) > 1e-3 for t, ok, ell in trace if ell < 0)
        assert nerr(xf[b], xo) < 5 * TOL
        acc += so["accepted"]; rej += so["rejected"]
    assert st["accepted"] == acc and st["rejected"] == rej and acc + rej > 10


def test_trajectory_with_more_drafts_than_transitions(free):
    """K larger than the whole schedule: every round drafts up to the last but one transition (the final, noise-free
    transition is never drafted) and the loop still matches the oracle."""
    sh, w, wd, model = _tiny_model(free)
    N, B, K, cfg = 6, 2, 9, 0.0
    sc = osched.make("linear", N)
    dsched = free.DeviceSchedule(free.linear_schedule(N))
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(24, 1, (B,) + shape)
    zt, zd = synth.normal(24, 2, (B, N) + shape), synth.normal(24, 3, (B, N) + shape)
    u = synth.uniform01(24, 4, (B, N)) * 1e-3                       # small uniforms: most drafts are accepted
    labels = np.array([0, 9], np.int32)
    xf, st = model.sample_trajectory(cu(x0), cu(labels, torch.int32), dsched, K, cfg, cu(zt), cu(zd), cu(u))
    acc = rej = calls = 0
    for b in range(B):
        xo, so, trace = _oracle_traj(sh, w, wd, sc, N, K, cfg, x0[b], int(labels[b]), zt[b], zd[b], u[b])
        assert all(abs(ell - np.log(u[b, t - 1])) > 1e-3 for t, ok, ell in trace if ell < 0)
        assert max(t for t, _, _ in trace) <= N - 1                 # the last transition is never verified as a draft
        assert nerr(xf[b], xo) < 5 * TOL
        acc += so["accepted"]; rej += so["rejected"]; calls += so["target_calls"]
    assert st["accepted"] == acc and st["rejected"] == rej and st["target_calls"] == calls
