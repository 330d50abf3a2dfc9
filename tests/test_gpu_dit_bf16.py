"""bf16 tensor-core mode against the fp64 oracle on bf16-representable weights.
Tolerance 2e-2 = max error / max |oracle| per output tensor (the bound stated for the bf16 mode of this library)."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit as odit, drafter as odrafter, schedule as osched
from gpu_util import cu, nerr

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def free():
    import paper_2511_20390_b200 as f
    f.lib()
    return f


def _model(free, sh, seed, depth=None, **kw):
    import dataclasses
    if depth is not None:
        sh = dataclasses.replace(sh, depth=depth)
    w = synth.make_target_weights(sh, seed, bf16=True, **kw)
    wd = synth.make_drafter_weights(sh, seed + 1, bf16=True, **kw)
    return sh, w, wd, free.Model(sh, w, wd, dtype="bf16")


@pytest.mark.parametrize("kw", [dict(), dict(ada_std=0.2, out_gain=2.0)])
def test_dit_s2_packed_pass(free, kw):
    # DiT-S/2 shaped: 4x32x32 latents (256 tokens), width 384, 12 blocks, 6 heads; B = 4 samples x K = 6 states
    sh, w, wd, model = _model(free, synth.DIT_S2, 11, **kw)
    N = 250
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    x, t, y = synth.pack_states(5, 4, 6, (sh.C, sh.H, sh.W), N, sh.n_classes)
    X, T, Y = x.reshape(24, sh.C, sh.H, sh.W), t.reshape(-1), y.reshape(-1)
    mean, eps, feat = model.dit_verify_pass(cu(X), cu(T, torch.int32), cu(Y, torch.int32), 0.0, dsched, want_eps=True, want_feat=True)
    torch.cuda.synchronize()
    pick = [0, 7, 13, 23]
    mo, eo, fo = odit.verify_pass(w, sh, sc, X[pick], T[pick], Y[pick], 0.0)
    errs = (nerr(eps[pick], eo), nerr(mean[pick], mo), nerr(feat[pick], fo))
    print("S/2 errors eps/mean/feat:", errs)
    assert max(errs) < TOL


def test_dit_s2_guided_and_drafter(free):
    sh, w, wd, model = _model(free, synth.DIT_S2, 21, depth=4, ada_std=0.2, out_gain=2.0)
    N = 250
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    n = 3
    x = synth.normal(8, 1, (n, sh.C, sh.H, sh.W))
    t, y = np.array([240, 100, 7], np.int32), np.array([1, 999, 400], np.int32)
    mean, eps, feat = model.dit_verify_pass(cu(x), cu(t, torch.int32), cu(y, torch.int32), 4.0, dsched, want_eps=True, want_feat=True)
    mo, eo, fo = odit.verify_pass(w, sh, sc, x, t, y, 4.0)
    assert max(nerr(eps, eo), nerr(mean, mo), nerr(feat, fo)) < TOL
    # drafter step from the oracle's features (rounded to bf16, as the GPU stores them)
    f_prev = synth.round_to_bf16(fo.astype(np.float32))
    z = synth.normal(8, 3, (n, sh.C, sh.H, sh.W))
    t2 = (t - 1).astype(np.int32)
    m_hat, x_hat, f_next = model.draft_step(cu(x), cu(f_prev, torch.bfloat16), cu(t2, torch.int32), cu(y, torch.int32), 4.0, dsched, cu(z))
    torch.cuda.synchronize()
    for i in range(n):
        mo_i, eo_i, fo_i = odrafter.guided_step(w, wd, sh, sc, x[i], f_prev[i], int(t2[i]), int(y[i]), 4.0)
        assert nerr(m_hat[i], mo_i) < TOL and nerr(f_next[i], fo_i) < TOL
        assert nerr(x_hat[i], mo_i + np.sqrt(sc.sigma2[t2[i]]) * z[i]) < TOL


def test_bf16_trajectory_bounding_regimes(free):
    # the sampling loop in bf16 mode on a small model, through the final statistics of an all-accept run, an
    # (almost) all-reject run and the plain sampler; single rounds are checked draft by draft in the teacher-forced tests
    import dataclasses
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=16)
    N, K, B = 12, 3, 2
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    shape = (sh.C, sh.H, sh.W)
    x0 = synth.normal(4, 1, (B,) + shape)
    zt, zd = synth.normal(4, 2, (B, N) + shape), synth.normal(4, 3, (B, N) + shape)
    labels = cu(np.array([3, 7], np.int32), torch.int32)
    w = synth.make_target_weights(sh, 1, bf16=True)
    wd = synth.make_drafter_weights(sh, 2, bf16=True)
    model = free.Model(sh, w, wd, dtype="bf16")
    # u = 0 accepts everything: rounds advance K+1 transitions
    xf, st = model.sample_trajectory(cu(x0), labels, dsched, K, 0.0, cu(zt), cu(zd), cu(np.zeros((B, N), np.float32)))
    assert st["rejected"] == 0 and st["accepted"] == st["draft_calls"] and torch.isfinite(xf).all()
    assert st["parallel_efficiency"] > 1.5
    # u = 1 with a random drafter rejects (almost) every first draft: two transitions per round
    xf2, st2 = model.sample_trajectory(cu(x0), labels, dsched, K, 0.0, cu(zt), cu(zd), cu(np.ones((B, N), np.float32)))
    assert st2["rejected"] >= st2["rounds"] // 2 and torch.isfinite(xf2).all()
    # K = 0: plain sampler, N target calls per sample
    xf3, st3 = model.sample_trajectory(cu(x0), labels, dsched, 0, 0.0, cu(zt))
    assert st3["target_calls"] == B * N


@pytest.mark.parametrize("cfg", [0.0, 3.0])
def test_round_teacher_forced_small(free, cfg):
    import dataclasses
    from gpu_util import check_round_teacher_forced
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32)
    w = synth.make_target_weights(sh, 5, bf16=True, ada_std=0.2, out_gain=2.0)
    wd = synth.make_drafter_weights(sh, 6, bf16=True, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, wd, dtype="bf16")
    n = check_round_teacher_forced(free, model, sh, 50, np.array([3, 10, 20, 30, 41], np.int64), np.array([1, 2, 3, 4, 5], np.int32), 4, cfg, 21)
    assert n.tolist() == [0, 1, 2, 3, 4]


def test_ragged_row_blocks_and_single_query_tile(free):
    # 3 sequences of 128 tokens: 384 rows = one and a half 256-row tiles of the CTA-pair GEMM (the second CTA of the
    # last pair has no rows), and an attention CTA with a single query tile
    import dataclasses
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32)
    w = synth.make_target_weights(sh, 31, bf16=True, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, None, dtype="bf16")
    N = 250
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    x = synth.normal(9, 1, (3, sh.C, sh.H, sh.W))
    t, y = np.array([200, 90, 3], np.int32), np.array([5, 77, 999], np.int32)
    mean, eps, feat = model.dit_verify_pass(cu(x), cu(t, torch.int32), cu(y, torch.int32), 0.0, dsched, want_eps=True, want_feat=True)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    mo, eo, fo = odit.verify_pass(w, sh, sc, x, t, y, 0.0)
    assert max(nerr(eps, eo), nerr(mean, mo), nerr(feat, fo)) < TOL


def test_rounds_as_cuda_graphs(free):
    """The rounds of a trajectory replayed as one CUDA graph (use_graph) and a round captured by the caller: both must
    reproduce the eager launches bit for bit (same kernels, same arguments, state in the workspace)."""
    import dataclasses
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32)
    N, K, B, cfg = 20, 3, 3, 2.0
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    shape = (sh.C, sh.H, sh.W)
    x0 = cu(synth.normal(4, 1, (B,) + shape))
    zt, zd = cu(synth.normal(4, 2, (B, N) + shape)), cu(synth.normal(4, 3, (B, N) + shape))
    u = cu(synth.uniform01(4, 4, (B, N)) * 1e-30)                    # a mix: tiny uniforms accept most drafts, not all
    labels = cu(np.array([3, 7, 11], np.int32), torch.int32)
    model = free.Model(sh, synth.make_target_weights(sh, 1, bf16=True), synth.make_drafter_weights(sh, 2, bf16=True), dtype="bf16")
    x_e, st_e = model.sample_trajectory(x0, labels, dsched, K, cfg, zt, zd, u)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        x_g, st_g = model.sample_trajectory(x0, labels, dsched, K, cfg, zt, zd, u, use_graph=True)
    torch.cuda.synchronize()
    assert st_e["rounds"] >= 3 and st_e["graph_rounds"] == 0 and st_g["graph_rounds"] == st_g["rounds"] - 1
    assert torch.equal(x_e, x_g) and {k: v for k, v in st_e.items() if k != "graph_rounds"} == {k: v for k, v in st_g.items() if k != "graph_rounds"}
    # the legacy default stream cannot be captured: the request is ignored there
    x_d, st_d = model.sample_trajectory(x0, labels, dsched, K, cfg, zt, zd, u, use_graph=True)
    assert torch.equal(x_e, x_d) and st_d["graph_rounds"] in (0, st_d["rounds"] - 1)
    # a round captured by the caller, after one eager call
    cursor = cu(np.array([2, 9, 15], np.int32), torch.int32)
    out = [torch.empty_like(x0), torch.empty_like(cursor), torch.zeros(B, dtype=torch.int32, device="cuda")]
    ref = [t.clone() for t in model.spec_round(x0, cursor, labels, dsched, K, cfg, zt, zd, u)]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            model.spec_round(x0, cursor, labels, dsched, K, cfg, zt, zd, u, x_next=out[0], cursor_next=out[1], n_accept=out[2])
    torch.cuda.synchronize()
    for _ in range(2):
        for t in out:
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(out, ref)) and model.device_error() == 0


def test_launch_overlap_does_not_change_results(free):
    """Programmatic dependent launch only moves a kernel's set-up ahead of its predecessor's end: with the switch on or off
    a packed pass over few token rows (where it is applied) gives the same bytes, eagerly and inside a captured round."""
    sh, w, wd, model = _model(free, synth.DIT_S2, 41, depth=3, ada_std=0.2, out_gain=2.0)
    N = 250
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    x, t, y = synth.pack_states(7, 2, 6, (sh.C, sh.H, sh.W), N, sh.n_classes)         # 12 states x 2 streams x 256 tokens = 6144 rows
    X, T, Y = cu(x.reshape(12, sh.C, sh.H, sh.W)), cu(t.reshape(-1), torch.int32), cu(y.reshape(-1), torch.int32)
    L = free.lib()
    try:
        assert L.free_set_launch_overlap(1) in (0, 1)
        on = [a.clone() for a in model.dit_verify_pass(X, T, Y, 4.0, dsched, want_eps=True, want_feat=True)]
        assert L.free_set_launch_overlap(0) == 1
        off = [a.clone() for a in model.dit_verify_pass(X, T, Y, 4.0, dsched, want_eps=True, want_feat=True)]
        torch.cuda.synchronize()
        assert model.device_error() == 0 and all(torch.equal(a, b) for a, b in zip(on, off))
    finally:
        L.free_set_launch_overlap(1)
