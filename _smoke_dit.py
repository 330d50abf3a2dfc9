"""Second half of the smoke check: a small bf16 packed pass and one speculative round, checked against the oracle."""
import dataclasses

import numpy as np
import torch


def smoke_dit():
    import synth
    import paper_2511_20390_b200 as free
    from oracle import dit as odit, schedule as osched, verify as overify

    sh = dataclasses.replace(synth.DIT_S2, depth=2, H=16, W=32)        # 128 tokens, width 384, 6 heads
    w = synth.make_target_weights(sh, 1, bf16=True, ada_std=0.2, out_gain=2.0)
    wd = synth.make_drafter_weights(sh, 2, bf16=True, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, wd, dtype="bf16")
    N = 50
    sc = osched.make("respaced", N)
    dsched = free.DeviceSchedule(free.respaced_schedule(N))
    cu = lambda a, dt=torch.float32: torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()
    x, t, y = synth.pack_states(3, 1, 4, (sh.C, sh.H, sh.W), N, sh.n_classes)
    mean, eps = model.dit_verify_pass(cu(x[0]), cu(t[0], torch.int32), cu(y[0], torch.int32), 4.0, dsched, want_eps=True)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    mo, eo, _ = odit.verify_pass(w, sh, sc, x[0, :2], t[0, :2], y[0, :2], 4.0)
    err = np.abs(eps[:2].cpu().numpy() - eo).max() / np.abs(eo).max()
    assert err < 2e-2, err
    # one speculative round; the verifier's decision is re-derived by the oracle from the round's own operands
    B, K, d = 2, 3, sh.d_latent
    x0 = cu(synth.normal(4, 1, (B, sh.C, sh.H, sh.W)))
    zt, zd = cu(synth.normal(4, 2, (B, N, d))), cu(synth.normal(4, 3, (B, N, d)))
    u = cu(synth.uniform01(4, 4, (B, N)))
    cursor = torch.ones(B, dtype=torch.int32, device="cuda")
    x_next, cur_next, n_acc = model.spec_round(x0, cursor, cu(y[0, :B], torch.int32), dsched, K, 0.0, zt, zd, u)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    assert torch.isfinite(x_next).all() and bool(((cur_next >= 2) & (cur_next <= 2 + K)).all())
    assert bool((cur_next == 2 + torch.clamp(n_acc + 1, max=K)).all())
