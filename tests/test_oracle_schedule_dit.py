"""Pins for the oracle's schedule and DiT layers: Gaussian-posterior algebra, library routines
(CPU torch, fp64), brute force, structural identities and the sizes the paper quotes."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth
from oracle import dit, schedule, drafter



# ----------------------------------------------------------------------------- schedule
def _golden():
    """key -> (value, tolerance) from tests/golden/paper_values.txt (the values the paper prints, each with its citation)."""
    import os
    out = {}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_values.txt")) as fh:
        for line in fh:
            line = line.split("#", 1)[0].split()
            if len(line) == 3:
                out[line[0]] = (float(line[1]), float(line[2]))
    return out


@pytest.mark.parametrize("kind,N", [("linear", 50), ("respaced", 250)])
def test_posterior_variance_is_the_gaussian_posterior(kind, N):
    # beta~ must be the variance of q(x_{t-1} | x_t, x_0): precision = alpha/beta + 1/(1 - abar_prev).
    sc = schedule.make(kind, N)
    abar_prev = np.concatenate([[1.0], sc.abar[:-1]])
    with np.errstate(divide="ignore"):
        prec = sc.alphas / sc.betas + 1.0 / (1.0 - abar_prev)
    assert np.allclose(sc.sigma2, 1.0 / prec, rtol=1e-12, atol=0)
    assert sc.sigma2[0] == 0.0 and np.all(sc.sigma2[1:] > 0)
    assert np.all(sc.sigma2 <= sc.betas + 1e-18)


@pytest.mark.parametrize("kind,N", [("linear", 50), ("respaced", 250)])
def test_mean_is_the_posterior_mean_for_the_true_noise(kind, N):
    # With x_t = sqrt(abar) x0 + sqrt(1-abar) eps, Eq. ddpm_update's mean equals the posterior mean
    # mu~(x_t, x0) = sqrt(abar_prev) beta/(1-abar) x0 + sqrt(alpha)(1-abar_prev)/(1-abar) x_t.
    sc = schedule.make(kind, N)
    rng = np.random.default_rng(0)
    x0, eps = rng.standard_normal(9), rng.standard_normal(9)
    for s in (0, 1, N // 2, N - 1):
        xt = np.sqrt(sc.abar[s]) * x0 + np.sqrt(1 - sc.abar[s]) * eps
        abar_prev = 1.0 if s == 0 else sc.abar[s - 1]
        mu = (np.sqrt(abar_prev) * sc.betas[s] / (1 - sc.abar[s]) * x0
              + np.sqrt(sc.alphas[s]) * (1 - abar_prev) / (1 - sc.abar[s]) * xt)
        assert np.allclose(sc.mean(xt, eps, s), mu, rtol=1e-11, atol=1e-12)
    assert np.allclose(sc.mean(x0, 0 * x0, 3), x0 / np.sqrt(sc.alphas[3]))


def _variance_after_chain(sc, s0_sq):
    """Variance of x_0 when data ~ N(0, s0_sq) and the chain runs with the EXACT noise prediction of that Gaussian
    (eps*(x, s) = sqrt(1 - abar_s) x / v_s, v_s = abar_s s0_sq + 1 - abar_s).  Also returns the largest relative
    gap to the forward marginals on the way."""
    v = sc.abar[-1] * s0_sq + 1.0 - sc.abar[-1]
    worst = 0.0
    for s in range(sc.N - 1, -1, -1):
        v_s = sc.abar[s] * s0_sq + 1.0 - sc.abar[s]
        gain = sc.coef_x[s] - sc.coef_eps[s] * np.sqrt(1.0 - sc.abar[s]) / v_s
        v = gain * gain * v + sc.sigma2[s]
        target = (sc.abar[s - 1] * s0_sq + 1.0 - sc.abar[s - 1]) if s > 0 else s0_sq
        worst = max(worst, abs(v / target - 1.0))
    return v, worst


@pytest.mark.parametrize("s0_sq", [0.25, 1.0, 4.0])
@pytest.mark.parametrize("eps", [0.0, 0.5, 1.0, 1.5])
def test_stochasticity_family_shares_the_marginals(eps, s0_sq):
    # Appendix "Stochasticity Hyperparameter": with the exact score every member of the family has the forward marginals
    # (up to the discretisation error of 1000 Euler-Maruyama steps)
    sc = schedule.Schedule(schedule.linear_betas(1000), stochasticity=eps)
    v, worst = _variance_after_chain(sc, s0_sq)
    assert abs(v / s0_sq - 1.0) < 0.03 and worst < 0.03


def test_stochasticity_special_members():
    b = schedule.linear_betas(100)
    ode = schedule.Schedule(b, stochasticity=0.0)
    assert np.all(ode.sigma2 == 0) and np.allclose(ode.coef_eps, 0.5 * b / np.sqrt(1 - ode.abar))      # probability-flow ODE
    sde, ddpm = schedule.Schedule(b, stochasticity=1.0), schedule.Schedule(b, variance="beta")
    # eps = 1 is the first-order (in beta) form of the DDPM step with sigma^2 = beta
    assert np.all(np.abs(sde.coef_x - ddpm.coef_x) <= b ** 2)
    assert np.allclose(sde.coef_eps, ddpm.coef_eps * np.sqrt(ddpm.alphas), rtol=1e-12)
    assert np.array_equal(sde.sigma2, ddpm.sigma2)
    two = schedule.Schedule(b, stochasticity=2.0)
    assert np.allclose(two.sigma2, 4 * sde.sigma2) and np.allclose(two.coef_eps, 2.5 * sde.coef_eps)


@pytest.mark.parametrize("variance", ["posterior", "beta", 0.3])
def test_fixed_variance_choices(variance):
    b = schedule.linear_betas(1000)
    sc, post, beta = schedule.Schedule(b, variance=variance), schedule.Schedule(b), schedule.Schedule(b, variance="beta")
    assert np.array_equal(sc.coef_x, post.coef_x) and np.array_equal(sc.coef_eps, post.coef_eps)     # only sigma changes
    assert sc.sigma2[0] == 0.0 and np.all(sc.sigma2[1:] >= post.sigma2[1:] * (1 - 1e-12)) and np.all(sc.sigma2[1:] <= b[1:] * (1 + 1e-12))
    if variance == 0.3:
        assert np.allclose(np.log(sc.sigma2[1:]), 0.3 * np.log(b[1:]) + 0.7 * np.log(post.sigma2[1:]))
        assert np.allclose(schedule.Schedule(b, variance=0.0).sigma2, post.sigma2) and np.allclose(schedule.Schedule(b, variance=1.0).sigma2[1:], b[1:])
    # any sigma between the two extremes keeps the marginals of unit-variance data (where beta is exact) within a few percent
    v, _ = _variance_after_chain(sc, 1.0)
    assert abs(v - 1.0) < 0.03


def test_library_schedule_tables_match_oracle():
    from paper_2511_20390_b200 import schedule as product
    for kw in ({}, {"variance": "beta"}, {"variance": 0.4}, {"stochasticity": 0.7}, {"stochasticity": 0.0}):
        for name, N in (("linear", 50), ("respaced", 250)):
            o = schedule.make(name, N, **kw)
            t = getattr(product, name + "_schedule")(N, **kw)
            for key in ("coef_x", "coef_eps", "sigma2", "t_embed_value"):
                assert np.allclose(t[key], getattr(o, key), rtol=1e-13, atol=0), (kw, name, key)


def test_respaced_keeps_abar_of_the_full_schedule():
    b, idx = schedule.respaced_betas(250)
    full = np.cumprod(1.0 - schedule.linear_betas(1000))
    assert idx[0] == 0 and idx[-1] == 999 and np.all(np.diff(idx) >= 4) and np.all(np.diff(idx) <= 5)
    assert np.allclose(np.cumprod(1.0 - b), full[idx], rtol=1e-12)
    assert np.array_equal(schedule.make("respaced", 250).t_embed_value, idx)
    lin = schedule.make("linear", 50)
    assert lin.betas[0] == 1e-4 and np.isclose(lin.betas[-1], 2e-2) and lin.abar[-1] < 0.62


# ----------------------------------------------------------------------------- layer primitives
def test_primitives_against_torch():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 48)) * 3 + 0.5
    t = torch.from_numpy(x)
    assert np.allclose(dit.layer_norm(x), F.layer_norm(t, (48,), eps=1e-6).numpy(), atol=1e-12)
    assert np.allclose(dit.gelu_tanh(x), F.gelu(t, approximate="tanh").numpy(), atol=1e-12)
    assert np.allclose(dit.silu(x), F.silu(t).numpy(), atol=1e-12)
    W, b = rng.standard_normal((5, 48)), rng.standard_normal(5)
    assert np.allclose(dit.linear(x, W, b), F.linear(t, torch.from_numpy(W), torch.from_numpy(b)).numpy(), atol=1e-12)


def test_attention_against_brute_force_and_torch():
    rng = np.random.default_rng(2)
    T, dh = 11, 6
    q, k, v = (rng.standard_normal((T, dh)) for _ in range(3))
    out = dit.attention(q, k, v)
    brute = np.zeros((T, dh))
    for i in range(T):
        wts = np.array([np.exp(sum(q[i, c] * k[j, c] for c in range(dh)) / np.sqrt(dh)) for j in range(T)])
        assert np.isclose((wts / wts.sum()).sum(), 1.0)
        for j in range(T):
            brute[i] += wts[j] / wts.sum() * v[j]
    assert np.allclose(out, brute, atol=1e-12)
    ref = F.scaled_dot_product_attention(*(torch.from_numpy(a)[None, None] for a in (q, k, v)))[0, 0].numpy()
    assert np.allclose(out, ref, atol=1e-12)


def test_multi_head_split_against_torch():
    rng = np.random.default_rng(3)
    T, D, h = 9, 24, 3
    x = rng.standard_normal((T, D))
    W, b = rng.standard_normal((3 * D, D)) * 0.2, rng.standard_normal(3 * D) * 0.1
    out = dit.multi_head_attention(x, W, b, h)
    qkv = F.linear(torch.from_numpy(x), torch.from_numpy(W), torch.from_numpy(b)).reshape(T, 3, h, D // h).permute(1, 2, 0, 3)
    ref = F.scaled_dot_product_attention(qkv[0][None], qkv[1][None], qkv[2][None])[0].permute(1, 0, 2).reshape(T, D)
    assert np.allclose(out, ref.numpy(), atol=1e-12)


def test_patch_embed_is_a_strided_convolution_and_unpatchify_inverts_layout():
    sh = synth.TINY
    w = synth.make_target_weights(sh, 5)
    x = synth.normal(5, 99, (sh.C, sh.H, sh.W)).astype(np.float64)
    tok = dit.linear(dit.patchify(x, sh), w["pe_w"], w["pe_b"])
    conv = F.conv2d(torch.from_numpy(x)[None], torch.from_numpy(w["pe_w"].astype(np.float64)).reshape(sh.D, sh.C, sh.patch, sh.patch),
                    torch.from_numpy(w["pe_b"].astype(np.float64)), stride=sh.patch)[0]
    assert np.allclose(tok, conv.flatten(1).T.numpy(), atol=1e-12)
    # unpatchify: token (i,j), entry (p,q,c) lands at channel c, pixel (i*P+p, j*P+q)
    g, P, co = sh.H // sh.patch, sh.patch, sh.c_out
    t = np.arange(sh.n_tok * sh.out_dim, dtype=np.float64).reshape(sh.n_tok, sh.out_dim)
    img = dit.unpatchify(t, sh)
    for (i, j, p, q, c) in [(0, 0, 0, 0, 0), (1, 2, 1, 0, 3), (3, 3, 1, 1, 7), (2, 0, 0, 1, 5)]:
        assert img[c, i * P + p, j * P + q] == t[i * g + j, (p * P + q) * co + c]


def test_timestep_features_and_position_table():
    f = dit.timestep_features(37.0, 256)
    assert f.shape == (256,) and np.isclose(f[0], np.cos(37.0)) and np.isclose(f[128], np.sin(37.0))
    assert np.isclose(f[127], np.cos(37.0 * 10000 ** (-127 / 128))) and np.allclose(f[:128] ** 2 + f[128:] ** 2, 1)
    pos = synth.pos_embed_2d(synth.TINY)
    assert pos.shape == (16, 64) and np.allclose(pos[0, :16], 0) and np.allclose(pos[0, 16:32], 1)
    assert np.isclose(pos[5, 0], np.sin(1.0), atol=1e-6) and np.isclose(pos[5, 32], np.sin(1.0), atol=1e-6)  # token 5 = (row 1, col 1)
    assert np.isclose(pos[6, 32], np.sin(2.0), atol=1e-6)


# ----------------------------------------------------------------------------- structure
def _tiny(seed=1, **kw):
    sh = synth.TINY
    return sh, synth.make_target_weights(sh, seed, **kw)


def test_zero_gates_make_blocks_the_identity():
    sh, w = _tiny()
    D = sh.D
    w = {k: v.copy() for k, v in w.items()}
    for j in (2, 5):                       # gate rows of the modulation regressor
        w["ada_w"][:, j * D:(j + 1) * D] = 0
        w["ada_b"][:, j * D:(j + 1) * D] = 0
    x = synth.normal(1, 50, (sh.C, sh.H, sh.W))
    _, f = dit.forward(w, sh, x, 10.0, 3)
    assert np.allclose(f, dit.embed(w, sh, x), atol=1e-14)


def test_zero_head_gives_zero_noise_and_scaled_state():
    sh, w = _tiny(out_gain=0.0)
    sc = schedule.make("linear", 50)
    x = synth.normal(1, 51, (1, sh.C, sh.H, sh.W))
    means, eps, _ = dit.verify_pass(w, sh, sc, x, [7], [2], 0.0)
    assert np.all(eps == 0) and np.allclose(means[0], x[0] / np.sqrt(sc.alphas[7]))


def test_block_against_torch_functional_ops():
    sh, w = _tiny(ada_std=0.3)
    W = dit._with_heads(w, sh)
    rng = np.random.default_rng(4)
    x, sc = rng.standard_normal((sh.n_tok, sh.D)), rng.standard_normal(sh.D)
    got = dit.block(x, sc, W, 1)
    T = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    xt, D, h = T(x), sh.D, sh.heads
    mod = F.linear(T(sc), T(w["ada_w"][1]), T(w["ada_b"][1])).chunk(6)
    hh = F.layer_norm(xt, (D,), eps=1e-6) * (1 + mod[1]) + mod[0]
    qkv = F.linear(hh, T(w["qkv_w"][1]), T(w["qkv_b"][1])).reshape(-1, 3, h, D // h).permute(1, 2, 0, 3)
    a = F.scaled_dot_product_attention(qkv[0][None], qkv[1][None], qkv[2][None])[0].permute(1, 0, 2).reshape(-1, D)
    xt = xt + mod[2] * F.linear(a, T(w["proj_w"][1]), T(w["proj_b"][1]))
    hh = F.layer_norm(xt, (D,), eps=1e-6) * (1 + mod[4]) + mod[3]
    hh = F.linear(F.gelu(F.linear(hh, T(w["fc1_w"][1]), T(w["fc1_b"][1])), approximate="tanh"), T(w["fc2_w"][1]), T(w["fc2_b"][1]))
    xt = xt + mod[5] * hh
    assert np.allclose(got, xt.numpy(), atol=1e-12)


def test_guidance_combination():
    sh, w = _tiny(ada_std=0.3, out_gain=5.0)
    x = synth.normal(1, 52, (sh.C, sh.H, sh.W))
    e_c, _ = dit.forward(w, sh, x, 20.0, 4)
    e_u, _ = dit.forward(w, sh, x, 20.0, sh.n_classes)
    assert np.abs(e_c - e_u).max() > 1e-6
    assert np.array_equal(dit.guided_eps(w, sh, x, 20.0, 4, 1.0)[0], e_c)
    e4, f = dit.guided_eps(w, sh, x, 20.0, 4, 4.0)
    assert np.allclose(e4, e_u + 4.0 * (e_c - e_u), atol=1e-15) and f.shape == (2, sh.n_tok, sh.D)


def test_packed_states_are_independent_sequences():
    sh, w = _tiny(ada_std=0.3)
    sc = schedule.make("linear", 50)
    x, t, y = synth.pack_states(3, 1, 4, (sh.C, sh.H, sh.W), 50, sh.n_classes)
    m_all, _, _ = dit.verify_pass(w, sh, sc, x[0], t[0], y[0], 0.0)
    m_one, _, _ = dit.verify_pass(w, sh, sc, x[0, 2:3], t[0, 2:3], y[0, 2:3], 0.0)
    assert np.array_equal(m_all[2], m_one[0]) and len(set(t[0].tolist())) == 4


# ----------------------------------------------------------------------------- sizes the paper quotes
def test_sizes_quoted_by_the_paper():
    xl = synth.DIT_XL2_512
    g = _golden()
    assert abs(xl.n_params() / 1e6 - g["target_params_millions"][0]) < g["target_params_millions"][1]
    assert g["drafter_params_millions_min"][0] * 1e6 < xl.drafter_params(1) < g["drafter_params_millions_max"][0] * 1e6
    assert xl.n_tok == g["feature_tokens"][0] and xl.D == g["feature_width"][0]
    assert abs(xl.n_tok * xl.D * 4 / 1e6 - g["feature_megabytes_fp32"][0]) < g["feature_megabytes_fp32"][1]
    ratio = xl.flops_per_sequence(depth=1) / xl.flops_per_sequence()
    assert np.isclose(ratio, 1 / g["drafter_cost_ratio_blocks"][0])
    assert abs(xl.flops_per_sequence() / 1e12 - 1.049) < 0.005


def test_drafter_reuses_target_embedding_and_is_one_block():
    sh, w = _tiny(ada_std=0.3)
    wd = synth.make_drafter_weights(sh, 9, ada_std=0.3)
    rng = np.random.default_rng(6)
    x, f = rng.standard_normal((sh.C, sh.H, sh.W)), rng.standard_normal((sh.n_tok, sh.D))
    eps, f_next = drafter.forward(w, wd, sh, x, f, 12.0, 1)
    # written out: fuse -> one block -> head
    g = np.concatenate([dit.embed(w, sh, x), f], axis=1) @ wd["fc_w"].astype(np.float64).T + wd["fc_b"]
    sc = dit.silu(dit.conditioning(w, sh, 12.0, 1))
    h = dit.block(g, sc, dit._with_heads(wd, sh), 0)
    assert np.allclose(f_next, h, atol=1e-14) and eps.shape == (sh.C, sh.H, sh.W)
    # the feature half of the fusion layer matters, and so does the latent half
    assert np.abs(drafter.forward(w, wd, sh, x, 0 * f, 12.0, 1)[1] - f_next).max() > 1e-3
    assert np.abs(drafter.forward(w, wd, sh, 0 * x, f, 12.0, 1)[1] - f_next).max() > 1e-3


# ----------------------------------------------------------------------------- conditioning, head, whole forward, guided drafter
_T = lambda a: torch.from_numpy(np.asarray(a, np.float64))


def _torch_conditioning(w, sh, tau, label):
    """c = W2 SiLU(W1 [cos, sin](tau w_i) + b1) + b2 + E[label], from torch functional ops only."""
    half = sh.freq_dim // 2
    ang = tau * torch.exp(-np.log(10000.0) * torch.arange(half, dtype=torch.float64) / half)
    feat = torch.cat([torch.cos(ang), torch.sin(ang)])
    e_t = F.linear(F.silu(F.linear(feat, _T(w["t_w1"]), _T(w["t_b1"]))), _T(w["t_w2"]), _T(w["t_b2"]))
    return e_t + F.embedding(torch.tensor(label), _T(w["y_emb"]))


def _torch_block(x, sc, w, i, h):
    D = x.shape[1]
    mod = F.linear(sc, _T(w["ada_w"][i]), _T(w["ada_b"][i])).chunk(6)
    y = F.layer_norm(x, (D,), eps=1e-6) * (1 + mod[1]) + mod[0]
    qkv = F.linear(y, _T(w["qkv_w"][i]), _T(w["qkv_b"][i])).reshape(-1, 3, h, D // h).permute(1, 2, 0, 3)
    a = F.scaled_dot_product_attention(qkv[0][None], qkv[1][None], qkv[2][None])[0].permute(1, 0, 2).reshape(-1, D)
    x = x + mod[2] * F.linear(a, _T(w["proj_w"][i]), _T(w["proj_b"][i]))
    y = F.layer_norm(x, (D,), eps=1e-6) * (1 + mod[4]) + mod[3]
    y = F.linear(F.gelu(F.linear(y, _T(w["fc1_w"][i]), _T(w["fc1_b"][i])), approximate="tanh"), _T(w["fc2_w"][i]), _T(w["fc2_b"][i]))
    return x + mod[5] * y


def _torch_head(x, sc, w, sh):
    """Modulated head, then fold: token (i, j) holds (row-in-patch, column-in-patch, channel)."""
    D, p, g = x.shape[1], sh.patch, sh.H // sh.patch
    shift, scale = F.linear(sc, _T(w["fada_w"]), _T(w["fada_b"])).chunk(2)
    tok = F.linear(F.layer_norm(x, (D,), eps=1e-6) * (1 + scale) + shift, _T(w["fin_w"]), _T(w["fin_b"]))
    # F.fold wants [C*kh*kw, L] with the channel slowest: reorder (p, q, c) -> (c, p, q)
    cols = tok.reshape(-1, p, p, sh.c_out).permute(3, 1, 2, 0).reshape(sh.c_out * p * p, g * g)
    return F.fold(cols[None], (sh.H, sh.W), kernel_size=p, stride=p)[0]


def test_conditioning_against_torch_functional_ops():
    sh, w = _tiny(seed=3)
    for tau, label in ((0.0, 0), (37.0, 4), (999.0, sh.n_classes)):         # the last one is the null-label row
        ref = _torch_conditioning(w, sh, tau, label).numpy()
        assert np.allclose(dit.conditioning(w, sh, tau, label), ref, rtol=0, atol=1e-13)
    # the two timestep layers really have a SiLU between them, and the label row really is added
    e = dit.conditioning(w, sh, 37.0, 4)
    assert np.abs(e - dit.conditioning(w, sh, 37.0, 5)).max() > 1e-3
    lin = dit.linear(dit.linear(dit.timestep_features(37.0, sh.freq_dim), w["t_w1"], w["t_b1"]), w["t_w2"], w["t_b2"])
    assert np.abs(e - (lin + w["y_emb"][4])).max() > 1e-4


def test_final_layer_against_torch_functional_ops():
    sh, w = _tiny(seed=4, ada_std=0.3, out_gain=2.0)
    rng = np.random.default_rng(8)
    x, sc = rng.standard_normal((sh.n_tok, sh.D)) * 2 + 0.3, rng.standard_normal(sh.D)
    got = dit.final_layer(x, sc, dit._with_heads(w, sh), sh)
    ref = _torch_head(_T(x), _T(sc), w, sh).numpy()
    assert got.shape == (sh.c_out, sh.H, sh.W) and np.allclose(got, ref, rtol=0, atol=1e-12)
    # the pin can tell shift from scale and sees the LayerNorm: each planted variant is far outside the tolerance
    D = sh.D
    mod = dit.linear(sc, w["fada_w"], w["fada_b"])
    swapped = dit.unpatchify(dit.linear(dit.layer_norm(x) * (1 + mod[:D]) + mod[D:], w["fin_w"], w["fin_b"]), sh)
    no_one = dit.unpatchify(dit.linear(dit.layer_norm(x) * mod[D:] + mod[:D], w["fin_w"], w["fin_b"]), sh)
    no_ln = dit.unpatchify(dit.linear(x * (1 + mod[D:]) + mod[:D], w["fin_w"], w["fin_b"]), sh)
    for wrong in (swapped, no_one, no_ln):
        assert np.abs(wrong - ref).max() > 1e-3


@pytest.mark.parametrize("label", [2, 10])
def test_whole_forward_against_torch_functional_ops(label):
    # conditioning -> embed (strided convolution) -> blocks -> modulated head -> fold -> first C channels
    sh, w = _tiny(seed=5, ada_std=0.3, out_gain=2.0)
    x = synth.normal(5, 60, (sh.C, sh.H, sh.W)).astype(np.float64)
    eps, feat = dit.forward(w, sh, x, 123.0, label)
    sc = F.silu(_torch_conditioning(w, sh, 123.0, label))
    h = F.conv2d(_T(x)[None], _T(w["pe_w"]).reshape(sh.D, sh.C, sh.patch, sh.patch), _T(w["pe_b"]), stride=sh.patch)[0]
    h = h.flatten(1).T + _T(w["pos"])
    for i in range(sh.depth):
        h = _torch_block(h, sc, w, i, sh.heads)
    out = _torch_head(h, sc, w, sh)
    assert np.allclose(feat, h.numpy(), rtol=0, atol=1e-12)
    assert eps.shape == (sh.C, sh.H, sh.W) and np.allclose(eps, out[:sh.C].numpy(), rtol=0, atol=1e-12)
    assert np.abs(eps).max() > 1e-2                                         # not a comparison of zeros


def test_guided_drafter_step_combines_two_streams_with_their_own_features():
    sh, w = _tiny(seed=6, ada_std=0.3, out_gain=3.0)
    wd = synth.make_drafter_weights(sh, 11, ada_std=0.3, out_gain=3.0)
    sc = schedule.make("linear", 50)
    rng = np.random.default_rng(12)
    x = rng.standard_normal((sh.C, sh.H, sh.W))
    f = rng.standard_normal((2, sh.n_tok, sh.D))
    s, label, cfg = 17, 3, 4.0
    m_hat, eps_hat, f_next = drafter.guided_step(w, wd, sh, sc, x, f, s, label, cfg)
    tau = sc.t_embed_value[s]
    e_c, f_c = drafter.forward(w, wd, sh, x, f[0], tau, label)               # conditional stream: label, its own feature
    e_u, f_u = drafter.forward(w, wd, sh, x, f[1], tau, sh.n_classes)        # unconditional stream: null label, its own feature
    eps_ref = e_u + cfg * (e_c - e_u)
    assert np.allclose(eps_hat, eps_ref, rtol=0, atol=1e-14)
    assert np.array_equal(f_next[0], f_c) and np.array_equal(f_next[1], f_u)
    assert np.allclose(m_hat, sc.coef_x[s] * x - sc.coef_eps[s] * eps_ref, rtol=0, atol=1e-13)   # Eq. ddpm_update
    assert np.allclose(m_hat, (x - sc.betas[s] / np.sqrt(1 - sc.abar[s]) * eps_ref) / np.sqrt(sc.alphas[s]), atol=1e-12)
    # swapping the two streams' features, guiding the other way round, or guiding the mean instead of the noise are all visible
    swapped = drafter.guided_step(w, wd, sh, sc, x, f[::-1], s, label, cfg)
    assert np.abs(swapped[1] - eps_hat).max() > 1e-3 and np.abs(swapped[2][0] - f_next[0]).max() > 1e-3
    assert np.abs((e_c + cfg * (e_u - e_c)) - eps_hat).max() > 1e-3
    # guidance off: one stream only, and the unconditional feature is not consulted
    m1, e1, f1 = drafter.guided_step(w, wd, sh, sc, x, f, s, label, 1.0)
    assert np.array_equal(e1, e_c) and f1.shape == (1, sh.n_tok, sh.D)
    # the drafter's whole forward against torch functional ops: fuse -> one block -> its own head
    g = F.linear(torch.cat([F.conv2d(_T(x)[None], _T(w["pe_w"]).reshape(sh.D, sh.C, sh.patch, sh.patch), _T(w["pe_b"]),
                                     stride=sh.patch)[0].flatten(1).T + _T(w["pos"]), _T(f[0])], dim=1), _T(wd["fc_w"]), _T(wd["fc_b"]))
    scc = F.silu(_torch_conditioning(w, sh, float(tau), label))
    hh = _torch_block(g, scc, wd, 0, sh.heads)
    assert np.allclose(f_c, hh.numpy(), atol=1e-12)
    assert np.allclose(e_c, _torch_head(hh, scc, wd, sh)[:sh.C].numpy(), atol=1e-12)
