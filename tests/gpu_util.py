"""Helpers shared by the GPU parity tests: oracle-side batches and the error measure."""
import numpy as np
import torch


def cu(a, dt=torch.float32):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()


def nerr(got, ref):
    """max_i |got_i - ref_i| / max_i |ref_i| (elementwise relative error is undefined near zeros)."""
    got = got.detach().float().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    ref = np.asarray(ref, np.float64)
    return float(np.abs(got.astype(np.float64).reshape(ref.shape) - ref).max() / max(np.abs(ref).max(), 1e-30))


def rms_rel(got, ref):
    """sqrt(mean (got - ref)^2) / sqrt(mean ref^2): unlike `nerr` it sees an error confined to small elements."""
    got = got.detach().float().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    ref = np.asarray(ref, np.float64)
    diff = got.astype(np.float64).reshape(ref.shape) - ref
    return float(np.sqrt(np.mean(diff * diff)) / max(np.sqrt(np.mean(ref * ref)), 1e-30))


def round_by_hand(free, model, sh, dsched, tables, x_cur, cursor, labels, K, cfg, zt, zd, u):
    """One round of Algorithm 1 assembled from the public calls (target step, K drafter steps, raw packed pass, fused
    verifier) for samples whose cursor leaves room for all K drafts.  x_cur [B,C,H,W], cursor [B] (1-based next
    transition), zt / zd [B,N,d], u [B,N]: numpy.  Returns a dict of numpy arrays, the verifier's operands included."""
    B, N = len(cursor), len(tables["sigma2"])
    shape = (sh.C, sh.H, sh.W)
    G = 2 if (cfg > 0 and cfg != 1.0) else 1
    i32 = lambda a: cu(np.asarray(a, np.int32), torch.int32)
    s_a = N - cursor                                               # schedule index of the target's own transition
    m_a, feat = model.dit_verify_pass(cu(x_cur), i32(s_a), i32(labels), cfg, dsched, want_feat=True)
    # x_a = m_a + sigma z from the library itself (a round without drafts is the target's own step): bf16 layers amplify
    # a last-bit difference of their input, so the host must not redo this arithmetic
    x_a = model.spec_round(cu(x_cur), i32(cursor), i32(labels), dsched, 0, cfg, cu(zt))[0].cpu().numpy()
    sig = np.sqrt(tables["sigma2"][s_a].astype(np.float32)).reshape(B, 1, 1, 1)
    assert nerr(x_a, m_a.cpu().numpy().astype(np.float64) + sig.astype(np.float64) * zt[np.arange(B), cursor - 1].reshape((B,) + shape)) < 1e-6
    x_prev, m_hat, x_hat = x_a, [], []
    for i in range(K):
        t = cursor + i + 1                                         # transition proposed by draft i
        mh, xh, feat = model.draft_step(cu(x_prev), feat, i32(N - t), i32(labels), cfg, dsched,
                                        cu(zd[np.arange(B), t - 1].reshape((B,) + shape)))
        m_hat.append(mh.cpu().numpy()); x_hat.append(xh.cpu().numpy())
        x_prev = x_hat[-1]
    m_hat, x_hat = np.stack(m_hat, 1), np.stack(x_hat, 1)          # [B,K,C,H,W]
    packed = np.concatenate([x_a[:, None], x_hat[:, :-1]], axis=1)
    t_pack = cursor[:, None] + 1 + np.arange(K)[None, :]
    s_pack = N - t_pack
    eps = model.dit_verify_pass_raw(cu(packed.reshape((B * K,) + shape)), i32(s_pack.reshape(-1)),
                                    i32(np.repeat(labels, K)), G == 2, dsched)
    cx, ce = tables["coef_x"][s_pack].astype(np.float32), tables["coef_eps"][s_pack].astype(np.float32)
    s2 = tables["sigma2"][s_pack].astype(np.float32)
    uu = u[np.arange(B)[:, None], t_pack - 1].astype(np.float32)
    x_out, n_acc, ell, means = free.spec_verify_fused(eps.reshape((B, K, G) + shape), cu(x_a), cu(m_hat), cu(x_hat), cu(cx), cu(ce),
                                                      cu(s2), cu(uu), cfg, want_logratio=True, want_means=True)
    torch.cuda.synchronize()
    return dict(x_a=x_a, m_hat=m_hat, x_hat=x_hat, means=means.cpu().numpy(), sigma2=s2, u=uu, ell=ell.cpu().numpy(),
                x_out=x_out.cpu().numpy(), n_acc=n_acc.cpu().numpy())


def check_round_teacher_forced(free, model, sh, N, cursor, labels, K, cfg, seed):
    """free_spec_round against (i) the same round assembled from the public calls and (ii) the oracle's verifier run on
    the GPU's own means (decisions cannot be compared with a pure-fp64 network: bf16 means move the log-ratio).  The
    uniforms are placed from a first pass (0 accepts, 1 rejects) so that the samples stop at different drafts."""
    import synth
    from oracle import verify as overify
    tables = free.respaced_schedule(N)
    dsched = free.DeviceSchedule(tables)
    B, d = len(cursor), sh.d_latent
    x_cur = synth.normal(seed, 1, (B, sh.C, sh.H, sh.W))
    zt, zd = synth.normal(seed, 2, (B, N, d)), synth.normal(seed, 3, (B, N, d))
    u = np.zeros((B, N), np.float32)
    for b in range(B):                                             # sample b accepts b drafts (mod K+1), then rejects
        stop = b % (K + 1)
        if stop < K:
            u[b, cursor[b] + stop] = 1.0                           # transition cursor + 1 + stop, 0-based column
    hand = round_by_hand(free, model, sh, dsched, tables, x_cur, cursor, labels, K, cfg, zt, zd, u)
    x1, c1, n1 = model.spec_round(cu(x_cur), cu(cursor, torch.int32), cu(labels, torch.int32), dsched, K, cfg, cu(zt), cu(zd), cu(u))
    torch.cuda.synchronize()
    assert model.device_error() == 0
    n1, c1, x1 = n1.cpu().numpy(), c1.cpu().numpy(), x1.cpu().numpy()
    assert np.array_equal(n1, hand["n_acc"])
    assert np.array_equal(c1, cursor + 1 + np.minimum(n1 + 1, K))
    assert nerr(x1, hand["x_out"]) < 1e-5
    # the oracle's verifier on the GPU's means, drafts and uniforms
    xo, no, ello = overify.spec_verify(hand["means"], hand["m_hat"], hand["x_hat"], hand["sigma2"], hand["u"])
    assert np.array_equal(no, n1)
    assert nerr(x1, xo) < 1e-5
    for b in range(B):
        k = min(int(n1[b]) + 1, K)
        assert np.allclose(hand["ell"][b, :k], ello[b, :k], rtol=1e-4, atol=1e-3)
    return n1
