"""Out-of-bounds guard: every kernel writes only inside the buffers it was given.  Outputs and the workspace are
embedded in larger allocations whose margins hold a sentinel byte; after the calls the margins must be intact.
(A stand-in for a memory checker: ragged shapes that leave partial tiles at every edge.)"""
import dataclasses

import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu
GUARD = 1 << 16           # bytes on each side


class Guarded:
    """A device buffer of `nbytes` with sentinel margins; `.t` is the usable part viewed as `dtype`."""
    def __init__(self, nbytes, dtype=torch.uint8, fill=None):
        self.n = nbytes
        self.raw = torch.full(((nbytes + 255) // 256 * 256 + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD:GUARD + nbytes].view(dtype)
        if fill is not None:
            self.t.copy_(fill.reshape(-1).view(dtype) if fill.dtype != dtype else fill.reshape(-1))

    def intact(self):
        return bool((self.raw[:GUARD] == 0xA5).all()) and bool((self.raw[GUARD + self.n:] == 0xA5).all())


@pytest.mark.parametrize("M,N,K", [(300, 320, 128), (2049, 1152, 256), (129, 192, 64), (777, 3456, 384), (1, 128, 64)])
def test_linear_outputs_stay_in_bounds(M, N, K):
    from paper_2511_20390_b200 import binding as b
    L = b.lib()
    g = torch.Generator(device="cuda"); g.manual_seed(M + N)
    A = torch.randn(M, K, generator=g, device="cuda", dtype=torch.float32).bfloat16()
    W = (torch.randn(N, K, generator=g, device="cuda", dtype=torch.float32) * 0.05).bfloat16()
    bias = torch.randn(N, generator=g, device="cuda", dtype=torch.float32)
    gate = torch.randn((M + 63) // 64, N, generator=g, device="cuda", dtype=torch.float32)
    ws = Guarded(256)
    st = torch.cuda.current_stream().cuda_stream
    for epi, od in ((b.EPI_BIAS, b.FREE_BF16), (b.EPI_BIAS, b.FREE_FP32), (b.EPI_BIAS_GELU, b.FREE_BF16), (b.EPI_GATE_RESIDUAL, b.FREE_FP32)):
        out = Guarded(M * N * (2 if od == b.FREE_BF16 else 4))
        resid = Guarded(M * N * 4, torch.float32, torch.zeros(M * N, device="cuda", dtype=torch.float32))
        ws.t.zero_()
        rc = L.free_op_linear(b.FREE_BF16, epi, od, M, N, K, A.data_ptr(), W.data_ptr(), bias.data_ptr(), out.t.data_ptr(),
                              resid.t.data_ptr(), gate.data_ptr(), gate.stride(0), 64, ws.t.data_ptr(), 256, st)
        assert rc == 0
        torch.cuda.synchronize()
        assert int(ws.t[:4].view(torch.int32).item()) == 0
        assert out.intact() and resid.intact() and ws.intact(), (epi, od)
        if epi == b.EPI_GATE_RESIDUAL:      # the whole residual was updated (no row or column skipped)
            ref = (A.float() @ W.float().T + bias) * gate.repeat_interleave(64, 0)[:M]
            assert (resid.t.view(M, N) - ref).abs().max().item() < 2e-2 * ref.abs().max().item()


def test_packed_pass_and_drafter_stay_in_workspace_and_outputs():
    import paper_2511_20390_b200 as free
    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32)          # 3 x 128 tokens = 384 rows: a ragged CTA-pair tile, single query tiles
    w = synth.make_target_weights(sh, 41, bf16=True, ada_std=0.2, out_gain=2.0)
    wd = synth.make_drafter_weights(sh, 42, bf16=True, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, wd, dtype="bf16")
    n = 3
    need = free.lib().free_workspace_bytes(model.ctx, n)
    ws = Guarded(need)
    model._ws = ws.t                                                       # exactly the size the library asked for
    N = 50
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    cu = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    x = cu(synth.normal(3, 1, (n, sh.C, sh.H, sh.W)))
    t, y = cu(np.array([40, 20, 1], np.int32), torch.int32), cu(np.array([1, 2, 3], np.int32), torch.int32)
    mean = Guarded(x.numel() * 4, torch.float32)
    out = model.dit_verify_pass(x, t, y, 0.0, dsched, want_feat=True, mean_out=mean.t.view(x.shape))
    feat = out[1]
    m_hat, x_hat, f_next = model.draft_step(x, feat, t, y, 0.0, dsched, cu(synth.normal(3, 2, (n, sh.C, sh.H, sh.W))))
    torch.cuda.synchronize()
    assert model.device_error() == 0
    assert ws.intact() and mean.intact()
    assert torch.isfinite(mean.t).all() and torch.isfinite(x_hat).all() and torch.isfinite(f_next.float()).all()


def test_verifier_stays_in_bounds():
    import paper_2511_20390_b200 as free
    B, K, d = 5, 7, 4096 + 4
    s2 = np.full((B, K), 0.02, np.float32)
    m, mh, xh, u = synth.verifier_inputs(77, B, K, d, 0.004, s2)
    cu = lambda a: torch.from_numpy(a).cuda()
    x_out = Guarded(B * d * 4, torch.float32)
    n_acc = Guarded(B * 4, torch.int32)
    free.spec_verify(cu(m), cu(mh), cu(xh), cu(s2), cu(u), x_out=x_out.t.view(B, d), n_accept=n_acc.t[:B])
    torch.cuda.synchronize()
    assert x_out.intact() and n_acc.intact()


def test_fused_verifier_stays_in_bounds():
    import paper_2511_20390_b200 as free
    B, K, G, shape = 5, 3, 2, (4, 32, 33)                  # d = 4224: ragged against the cluster stride
    d = int(np.prod(shape))
    eps, x_first, mh, xh, u = synth.eps_verifier_inputs(4, B, K, G, shape, 0.01, np.full((B, K), 0.02), eps_std=0.1)
    cu = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).cuda()
    one = torch.ones(B, K, device="cuda", dtype=torch.float32)
    x_out, means, n_acc = Guarded(B * d * 4, torch.float32), Guarded(B * K * d * 4, torch.float32), Guarded(B * 4, torch.int32)
    ell, d2 = Guarded(B * K * 4, torch.float32), Guarded(B * K * 4, torch.float32)
    L = free.lib()
    st = torch.cuda.current_stream().cuda_stream
    ts = [cu(eps), cu(x_first), cu(mh), cu(xh)]
    ce, s2, uu = 0.05 * one, 0.02 * one, cu(u)
    for chunk in (0, 2):
        rc = L.spec_verify_fused(B, K, d, G, 4.0, ts[0].data_ptr(), ts[1].data_ptr(), ts[2].data_ptr(), ts[3].data_ptr(),
                                 one.data_ptr(), ce.data_ptr(), s2.data_ptr(), None, uu.data_ptr(), None, chunk,
                                 x_out.t.data_ptr(), n_acc.t.data_ptr(), ell.t.data_ptr(), d2.t.data_ptr(), means.t.data_ptr(), st)
        assert rc == 0
        torch.cuda.synchronize()
        assert x_out.intact() and means.intact() and n_acc.intact() and ell.intact() and d2.intact()
