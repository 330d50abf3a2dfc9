"""spec_verify_fused (CUDA: guidance + Eq. ddpm_update + Algorithm 2 from the packed pass's noise predictions) against
the oracle on identical fp32 inputs, and the raw packed pass + fused verifier against the two-step path."""
import dataclasses

import numpy as np
import pytest
import torch

import synth
from gpu_util import cu, nerr
from oracle import schedule as osched
from oracle import verify as overify

pytestmark = pytest.mark.gpu

TOL_ELL = 1e-4          # decisions may differ only where |ell - log u| is below this


def _inputs(seed, B, K, shape, G, s_rel=1.0, sigma2=0.02, eps_std=1.0, ce=0.05):
    """Inputs with |m_hat - m| of the order of s_rel * sigma: coef_x is 1 up to 1e-4, so the mean is the packed state
    minus a small multiple of eps, and the draft means sit s away from the packed state."""
    d = int(np.prod(shape))
    s2 = np.full((B, K), sigma2, np.float32) if np.isscalar(sigma2) else np.asarray(sigma2, np.float32)
    sig = float(np.sqrt(s2.mean()))
    s = s_rel * sig / np.sqrt(d)
    eps, x_first, m_hat, x_hat, u = synth.eps_verifier_inputs(seed, B, K, G, shape, s, s2, eps_std=eps_std * s / ce)
    coef_x = (1.0 + 1e-4 * s_rel * sig / np.sqrt(d) * np.linspace(-1, 1, B * K)).astype(np.float32).reshape(B, K)
    coef_eps = np.full((B, K), ce, np.float32)
    return dict(eps=eps, x_first=x_first, m_hat=m_hat, x_hat=x_hat, u=u, s2=s2, cx=coef_x, ce=coef_eps)


def _run(i, w_cfg, lam=None, n_valid=None, chunk=0):
    import paper_2511_20390_b200 as free
    x, n, ell, means = free.spec_verify_fused(cu(i["eps"]), cu(i["x_first"]), cu(i["m_hat"]), cu(i["x_hat"]), cu(i["cx"]), cu(i["ce"]),
                                              cu(i["s2"]), cu(i["u"]), w_cfg, lam=cu(lam), n_valid=cu(n_valid, torch.int32),
                                              chunk=chunk, want_logratio=True, want_means=True)
    torch.cuda.synchronize()
    return x.cpu().numpy(), n.cpu().numpy(), ell.cpu().numpy(), means.cpu().numpy()


def _dist2(i, w_cfg, chunk=0):
    import paper_2511_20390_b200 as free
    out = free.spec_verify_fused(cu(i["eps"]), cu(i["x_first"]), cu(i["m_hat"]), cu(i["x_hat"]), cu(i["cx"]), cu(i["ce"]),
                                 cu(i["s2"]), cu(i["u"]), w_cfg, chunk=chunk, want_logratio=True, want_dist2=True)
    torch.cuda.synchronize()
    return out[1].cpu().numpy(), out[2].cpu().numpy(), out[3].cpu().numpy()


def _compare(i, w_cfg, lam=None, n_valid=None, chunk=0):
    B, K = i["u"].shape
    x, n, ell, means = _run(i, w_cfg, lam, n_valid, chunk)
    xo, no, ello, mo = overify.spec_verify_from_eps(i["eps"], i["x_first"], i["m_hat"], i["x_hat"], i["cx"], i["ce"], w_cfg,
                                                    i["s2"], i["u"], lam, n_valid)
    nv = np.full(B, K) if n_valid is None else n_valid
    lam_ = np.ones((B, K)) if lam is None else lam
    n_exempt = 0
    for b in range(B):
        # drafts examined by the kernel: all present ones, or whole chunks up to the one with the first rejection
        seen = nv[b] if chunk == 0 else min(nv[b], (min(n[b], nv[b] - 1) // chunk + 1) * chunk) if nv[b] else 0
        ell_o = np.array([overify.log_ratio(i["x_hat"][b, k], mo[b, k], i["m_hat"][b, k], float(i["s2"][b, k]), float(lam_[b, k]))
                          for k in range(seen)])
        if seen:
            assert np.allclose(ell[b, :seen], ell_o, rtol=2e-6, atol=1e-6), (b, ell[b, :seen], ell_o)
            assert np.abs(means[b, :seen] - mo[b, :seen]).max() <= 2e-7 * np.abs(mo[b, :seen]).max()
        assert np.all(np.isnan(ell[b, seen:]))
        if n[b] != no[b]:
            k = min(n[b], no[b])
            assert abs(ell_o[k] - np.log(float(i["u"][b, k]))) < TOL_ELL, (b, k, ell_o[k], i["u"][b, k])
            n_exempt += 1
            continue
        if nv[b] == 0:
            assert np.all(x[b] == 0)
            continue
        assert np.abs(x[b] - xo[b]).max() <= 1e-5 * np.abs(xo[b]).max() + 1e-7, b
    assert n_exempt <= max(1, B // 50)
    return n, no


CASES = [
    # latent shape, G, B, K
    ((4, 64, 64), 2, 3, 6),          # the 512^2 latent: cluster of 8
    ((4, 32, 32), 1, 5, 16),         # 256^2 latent, no guidance: cluster of 4
    ((3, 12, 20), 2, 4, 4),          # d = 720: single CTA
    ((2, 9, 15), 2, 3, 5),           # d = 270: not a multiple of 4, scalar loads
    ((4, 32, 33), 2, 2, 3),          # d = 4224: multiple of 4, ragged against the cluster stride
    ((1, 1, 6), 1, 9, 3),            # tiny state
    ((4097,), 2, 2, 5),              # odd length above the clustered threshold
    ((4, 64, 64), 2, 2, 33),         # K = 33
    ((4, 192, 192), 2, 1, 3),        # large latent
    ((4, 64, 64), 2, 200, 2),        # batch wide enough to narrow the clusters
    ((4, 16, 16), 2, 2, 64),         # the largest K
]


@pytest.mark.parametrize("shape,G,B,K", CASES)
def test_matches_oracle(shape, G, B, K):
    i = _inputs(11 + B + K, B, K, shape, G, s_rel=1.0)
    n, no = _compare(i, 4.0)
    assert n.min() >= 0 and n.max() <= K


def test_mixed_decisions_relaxed_ragged_and_early_exit():
    shape, G, B, K = (4, 32, 32), 2, 48, 8
    i = _inputs(5, B, K, shape, G, s_rel=0.6)
    n, _ = _compare(i, 1.5)
    assert 0 < n.sum() < B * K and len(set(n.tolist())) >= 3
    lam = np.tile(synth.lambda_profile(K, floor=0.05, knee=0.5), (B, 1))
    n_rel, _ = _compare(i, 1.5, lam=lam)
    assert n_rel.sum() > n.sum() and np.all(n_rel >= n)
    nv = (np.arange(B) % (K + 1)).astype(np.int32)
    n_r, _ = _compare(i, 1.5, n_valid=nv)
    assert np.all(n_r <= nv)
    # early exit: same decisions and states, log-ratios only for the chunks that were read
    x0, n0, ell0, _ = _run(i, 1.5)
    for chunk in (1, 3, 4, 8, 11):
        _compare(i, 1.5, chunk=chunk)
        xc, nc2, ellc, _ = _run(i, 1.5, chunk=chunk)
        assert np.array_equal(nc2, n0) and np.array_equal(xc, x0)
        seen = ~np.isnan(ellc)
        assert np.array_equal(ellc[seen], ell0[seen])
        for b in range(B):
            assert seen[b].sum() == min(K, (min(n0[b], K - 1) // chunk + 1) * chunk)
    n_rc, _ = _compare(i, 1.5, n_valid=nv, chunk=3)
    assert np.array_equal(n_rc, n_r)


def test_mean_distance_output():
    # |m_hat - m|^2 per examined draft, against the oracle's means; NaN exactly where the log-ratio is NaN
    shape, G, B, K = (4, 32, 32), 2, 6, 8
    i = _inputs(31, B, K, shape, G, s_rel=0.6)
    mo = np.stack([overify.means_from_stream_eps(i["eps"][b], i["x_first"][b], i["x_hat"][b], i["cx"][b], i["ce"][b], 1.5) for b in range(B)])
    ref = ((i["m_hat"].astype(np.float64) - mo) ** 2).sum(axis=(2, 3, 4))
    for chunk in (0, 2):
        n, ell, d2 = _dist2(i, 1.5, chunk)
        seen = ~np.isnan(ell)
        assert np.array_equal(np.isnan(d2), ~seen) and (chunk > 0 or seen.all())
        assert np.allclose(d2[seen], ref[seen], rtol=1e-6)


def test_degenerate_cases():
    shape, G, B, K = (4, 16, 16), 2, 4, 3
    i = _inputs(9, B, K, shape, G, s_rel=30.0)
    # u = 0 accepts everything: the state is the last draft
    j = dict(i, u=np.zeros((B, K), np.float32))
    x, n, _, _ = _run(j, 4.0)
    assert np.all(n == K) and np.array_equal(x, i["x_hat"][:, -1])
    # far-off drafts with u = 1: the first draft is rejected; the reflection preserves the two norms (Lemma 2)
    j = dict(i, u=np.ones((B, K), np.float32))
    x, n, _, means = _run(j, 4.0)
    assert np.all(n == 0)
    for b in range(B):
        m0, mh0, xh0 = means[b, 0].astype(np.float64), i["m_hat"][b, 0], i["x_hat"][b, 0]
        assert np.isclose(np.linalg.norm(x[b] - m0), np.linalg.norm(xh0 - mh0), rtol=1e-5)
        assert np.isclose(np.linalg.norm(x[b] - mh0), np.linalg.norm(xh0 - m0), rtol=1e-5)
    # a non-positive variance is reported per sample and leaves x_out untouched
    bad = i["s2"].copy(); bad[1, 0] = 0.0; bad[2, 2] = np.nan
    x, n, _, _ = _run(dict(i, s2=bad, u=np.zeros((B, K), np.float32)), 4.0)
    assert n[1] == -5 and n[2] == -5 and n[0] == K and n[3] == K and np.all(x[1] == 0) and np.all(x[2] == 0)
    # with the early exit a bad variance behind the first rejection is never looked at
    x, n, _, _ = _run(dict(i, s2=bad, u=np.ones((B, K), np.float32)), 4.0, chunk=1)
    assert n[1] == -5 and n[2] == 0 and n[0] == 0


def test_argument_errors():
    import paper_2511_20390_b200 as free
    i = _inputs(3, 2, 2, (4, 16, 16), 2)
    with pytest.raises(free.FreeError):
        _run(i, 4.0, chunk=-1)
    with pytest.raises(free.FreeError):                     # three streams
        _run(dict(i, eps=np.concatenate([i["eps"], i["eps"][:, :, :1]], axis=2)), 4.0)
    L = free.lib()
    assert L.spec_verify_fused(1, 0, 16, 1, 1.0, *([None] * 10), 0, *([None] * 6)) != 0
    t = cu(np.zeros(16, np.float32))
    p = t.data_ptr()
    assert L.spec_verify_fused(0, 2, 8, 1, 1.0, p, p, p, p, p, p, p, None, p, None, 0, p, p, None, None, None, None) == 0      # empty batch
    assert L.spec_verify_fused(1, 65, 8, 1, 1.0, p, p, p, p, p, p, p, None, p, None, 0, p, p, None, None, None, None) == -2    # K too large


def test_full_size_point_sampled_against_oracle():
    # the benchmark's fused-verifier workload (K = 16, B = 256, 4x64x64 latents, guidance): a sample of the batch
    shape, G, B, K = (4, 64, 64), 2, 256, 16
    sc = osched.make("respaced", 250)
    s2 = np.tile(sc.sigma2[np.linspace(240, 20, K).astype(int)].astype(np.float32), (B, 1))
    i = _inputs(21, B, K, shape, G, s_rel=0.35, sigma2=s2)
    x, n, ell, _ = _run(i, 4.0)
    pick = [0, 1, 77, 128, 255]
    sub = {k: v[pick] for k, v in i.items()}
    xo, no, _, _ = overify.spec_verify_from_eps(sub["eps"], sub["x_first"], sub["m_hat"], sub["x_hat"], sub["cx"], sub["ce"], 4.0,
                                                sub["s2"], sub["u"])
    assert np.array_equal(n[pick], no)
    assert np.abs(x[pick] - xo).max() <= 1e-5 * np.abs(xo).max()
    assert 0 < n.sum() < B * K
    logu = np.log(i["u"].astype(np.float64))
    for b in range(B):
        assert np.all(logu[b, :n[b]] <= np.minimum(0, ell[b, :n[b]]) + 1e-3)
        if n[b] < K:
            assert logu[b, n[b]] > min(0, ell[b, n[b]]) - 1e-3
    xe, ne, _, _ = _run(i, 4.0, chunk=4)
    assert np.array_equal(ne, n) and np.array_equal(xe, x)


@pytest.mark.parametrize("dtype,cfg", [("fp32", 0.0), ("fp32", 3.0), ("bf16", 3.0)])
def test_raw_pass_plus_fused_verifier_equals_two_step_path(dtype, cfg):
    """dit_verify_pass_raw + spec_verify_fused against dit_verify_pass + spec_verify on a small model: the same
    network output reaches the verifier through both routes."""
    import paper_2511_20390_b200 as free
    bf = dtype == "bf16"
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32) if bf else synth.TINY
    w = synth.make_target_weights(sh, 31, bf16=bf, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, None, dtype=dtype)
    N, B, K = 50, 3, 4
    tables = free.respaced_schedule(N)
    dsched = free.DeviceSchedule(tables)
    shape = (sh.C, sh.H, sh.W)
    t_idx = np.tile(np.arange(40, 40 - K, -1, dtype=np.int32), (B, 1))
    labels = np.tile(np.arange(B, dtype=np.int32)[:, None], (1, K))
    s2 = tables["sigma2"][t_idx].astype(np.float32)
    i = _inputs(17, B, K, shape, 1, s_rel=1.0, sigma2=s2)
    packed = np.concatenate([i["x_first"][:, None], i["x_hat"][:, :-1]], axis=1)          # (x_a, first K-1 drafts)
    flat = lambda a: cu(a.reshape((B * K,) + a.shape[2:]))
    G = 2 if cfg > 0 else 1
    mean = model.dit_verify_pass(flat(packed), cu(t_idx.reshape(-1), torch.int32), cu(labels.reshape(-1), torch.int32), cfg, dsched)
    eps = model.dit_verify_pass_raw(flat(packed), cu(t_idx.reshape(-1), torch.int32), cu(labels.reshape(-1), torch.int32), cfg > 0, dsched)
    assert model.device_error() == 0
    mean = mean.reshape((B, K) + mean.shape[1:])
    # draft means placed so that every log-ratio is about -2: with r = x_hat - m_hat = g * (sign-flipped (x_hat - m)),
    # ell = (|r|^2 - |x_hat - m|^2) / (2 sigma^2) = (g^2 - 1) |x_hat - m|^2 / (2 sigma^2)
    diff = i["x_hat"].astype(np.float64) - mean.cpu().numpy()
    flip = np.where(synth.normal(5, 1, diff.shape[2:]) > 0, 1.0, -1.0)
    g = np.sqrt(1.0 - 4.0 * s2.astype(np.float64) / (diff ** 2).sum(axis=(2, 3, 4)))
    mh = (i["x_hat"] - g[:, :, None, None, None] * flip * diff).astype(np.float32)
    xh = i["x_hat"]
    cx, ce = tables["coef_x"][t_idx].astype(np.float32), tables["coef_eps"][t_idx].astype(np.float32)
    # uniforms placed half a unit of log-ratio on either side of the threshold, so that decisions are mixed and robust
    _, _, ell0 = free.spec_verify(mean.contiguous(), cu(mh), cu(xh), cu(s2), cu(np.ones((B, K), np.float32)), want_logratio=True)
    side = np.where((np.arange(B)[:, None] + np.arange(K)[None, :]) % 2 == 1, 0.5, -0.5)
    u = np.clip(np.exp(ell0.cpu().numpy().astype(np.float64) + side), 1e-30, 1.0).astype(np.float32)
    x1, n1, ell1 = free.spec_verify(mean.contiguous(), cu(mh), cu(xh), cu(s2), cu(u), want_logratio=True)
    x2, n2, ell2, means2 = free.spec_verify_fused(eps.reshape((B, K, G) + shape), cu(i["x_first"]), cu(mh), cu(xh),
                                                  cu(cx), cu(ce), cu(s2), cu(u), cfg, want_logratio=True, want_means=True)
    torch.cuda.synchronize()
    assert nerr(means2, mean.cpu().numpy()) < 1e-6
    assert np.allclose(ell1.cpu().numpy(), ell2.cpu().numpy(), rtol=1e-3, atol=2e-3)
    assert np.array_equal(n1.cpu().numpy(), n2.cpu().numpy())
    assert 0 < int(n1.sum()) < B * K
    assert nerr(x2, x1.cpu().numpy()) < 1e-5


def test_raw_pass_streams_match_oracle_forward():
    """dit_verify_pass_raw returns the noise prediction of each stream as an image: conditional stream = the oracle's
    forward with the label, unconditional stream = with the null label (un-patchify fused into the head's store)."""
    import paper_2511_20390_b200 as free
    from oracle import dit as odit
    sh = dataclasses.replace(synth.TINY, H=8, W=12)                 # non-square grid: 4 x 6 tokens
    w = synth.make_target_weights(sh, 3, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, None, dtype="fp32")
    tables = free.respaced_schedule(50)
    dsched = free.DeviceSchedule(tables)
    x = synth.normal(8, 1, (2, sh.C, sh.H, sh.W))
    t = np.array([40, 7], np.int32); y = np.array([1, 5], np.int32)
    eps = model.dit_verify_pass_raw(cu(x), cu(t, torch.int32), cu(y, torch.int32), True, dsched)
    e1 = model.dit_verify_pass_raw(cu(x), cu(t, torch.int32), cu(y, torch.int32), False, dsched)
    torch.cuda.synchronize()
    assert tuple(eps.shape) == (2, 2, sh.C, sh.H, sh.W) and tuple(e1.shape) == (2, 1, sh.C, sh.H, sh.W)
    for n in range(2):
        tau = float(tables["t_embed_value"][t[n]])
        ref_c, _ = odit.forward(w, sh, x[n], tau, int(y[n]))
        ref_u, _ = odit.forward(w, sh, x[n], tau, sh.n_classes)
        assert nerr(eps[n, 0], ref_c) < 1e-4 and nerr(eps[n, 1], ref_u) < 1e-4 and nerr(e1[n, 0], ref_c) < 1e-4
