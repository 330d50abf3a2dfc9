"""Target DiT forward in fp64, one sequence at a time (TEST INFRASTRUCTURE ONLY).

The paper uses DiT-XL/2 as published and does not restate it (Sec. 3.1, Sec. 4);
the layer definitions below are the adaLN-Zero DiT block: timestep + class
conditioning c, per-block (shift, scale, gate) x 2 regressed from SiLU(c),
LayerNorm without affine parameters, multi-head self-attention over all tokens,
GELU(tanh) MLP of ratio 4, and a modulated final projection back to patches.
The "top-block feature" f is the token matrix after the last block (Sec. 3.1,
Fig. top_block).  Weight dict layout: see synth.models.
"""
import numpy as np

LN_EPS = 1e-6


def silu(a):
    return a / (1.0 + np.exp(-a))


def gelu_tanh(a):
    return 0.5 * a * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (a + 0.044715 * a ** 3)))


def layer_norm(x):
    """Normalise each row to zero mean / unit (biased) variance; no affine."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + LN_EPS)


def linear(x, W, b):
    return x @ np.asarray(W, np.float64).T + np.asarray(b, np.float64)


def timestep_features(tau: float, freq_dim: int):
    """[cos(tau w_i), sin(tau w_i)], w_i = 10000^(-i/half), i < half = freq_dim/2."""
    half = freq_dim // 2
    w = np.exp(-np.log(10000.0) * np.arange(half, dtype=np.float64) / half)
    a = float(tau) * w
    return np.concatenate([np.cos(a), np.sin(a)])


def conditioning(w, shape, tau: float, label: int):
    """c = MLP(features(tau)) + E[label]; label == n_classes selects the null class."""
    h = silu(linear(timestep_features(tau, shape.freq_dim), w["t_w1"], w["t_b1"]))
    e_t = linear(h, w["t_w2"], w["t_b2"])
    return e_t + np.asarray(w["y_emb"][label], np.float64)


def patchify(x, shape):
    """[C,H,W] -> [n_tok, C*p*p]; token order row-major over the patch grid, vector
    order (channel, row-in-patch, column-in-patch)."""
    C, H, W, p = shape.C, shape.H, shape.W, shape.patch
    x = np.asarray(x, np.float64).reshape(C, H // p, p, W // p, p)
    return x.transpose(1, 3, 0, 2, 4).reshape(shape.n_tok, C * p * p)


def unpatchify(tok, shape):
    """[n_tok, c_out*p*p] -> [c_out,H,W]; vector order (row-in-patch, column-in-patch, channel)."""
    H, W, p, co = shape.H, shape.W, shape.patch, shape.c_out
    t = tok.reshape(H // p, W // p, p, p, co)
    return t.transpose(4, 0, 2, 1, 3).reshape(co, H, W)


def embed(w, shape, x):
    """Patch embedding plus the fixed position table."""
    return linear(patchify(x, shape), w["pe_w"], w["pe_b"]) + np.asarray(w["pos"], np.float64)


def attention(q, k, v):
    """softmax(q k^T / sqrt(d_h)) v for one head; q,k,v are [n_tok, d_h]."""
    s = (q @ k.T) / np.sqrt(q.shape[1])
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v


def multi_head_attention(h, Wqkv, bqkv, heads):
    """qkv = W h + b, split along the output as (3, heads, d_h); heads are concatenated back."""
    T, D = h.shape
    dh = D // heads
    qkv = linear(h, Wqkv, bqkv).reshape(T, 3, heads, dh)
    out = np.empty((T, D), dtype=np.float64)
    for a in range(heads):
        out[:, a * dh:(a + 1) * dh] = attention(qkv[:, 0, a], qkv[:, 1, a], qkv[:, 2, a])
    return out


def block(x, sc, W, i):
    """One adaLN-Zero block.  `sc` = SiLU(c); `W` holds the stacked block weights; i = block index.
    x <- x + g1 * proj(MHA(LN(x)(1+s1)+b1));  x <- x + g2 * fc2(GELU(fc1(LN(x)(1+s2)+b2)))."""
    D = x.shape[1]
    mod = linear(sc, W["ada_w"][i], W["ada_b"][i])
    b1, s1, g1, b2, s2, g2 = (mod[j * D:(j + 1) * D] for j in range(6))
    h = layer_norm(x) * (1.0 + s1) + b1
    a = multi_head_attention(h, W["qkv_w"][i], W["qkv_b"][i], W["_heads"])
    x = x + g1 * linear(a, W["proj_w"][i], W["proj_b"][i])
    h = layer_norm(x) * (1.0 + s2) + b2
    h = gelu_tanh(linear(h, W["fc1_w"][i], W["fc1_b"][i]))
    x = x + g2 * linear(h, W["fc2_w"][i], W["fc2_b"][i])
    return x


def final_layer(x, sc, W, shape):
    """(b, s) = W_ada SiLU(c); out = W (LN(x)(1+s)+b); returns the image-shaped output [c_out,H,W]."""
    D = x.shape[1]
    mod = linear(sc, W["fada_w"], W["fada_b"])
    b, s = mod[:D], mod[D:]
    out = linear(layer_norm(x) * (1.0 + s) + b, W["fin_w"], W["fin_b"])
    return unpatchify(out, shape)


def _with_heads(w, shape):
    W = dict(w)
    W["_heads"] = shape.heads
    return W


def forward(w, shape, x, tau: float, label: int, depth=None):
    """One sequence through the target.  Returns (eps [C,H,W], feature [n_tok,D])."""
    W = _with_heads(w, shape)
    sc = silu(conditioning(w, shape, tau, label))
    h = embed(w, shape, x)
    for i in range(shape.depth if depth is None else depth):
        h = block(h, sc, W, i)
    out = final_layer(h, sc, W, shape)
    return out[:shape.C], h


def guided_eps(w, shape, x, tau: float, label: int, cfg_scale: float):
    """Classifier-free guidance: eps = eps_u + w (eps_c - eps_u); cfg_scale <= 0 or == 1 disables
    it.  Returns (eps, features) with features stacked as [G, n_tok, D], conditional first."""
    eps_c, f_c = forward(w, shape, x, tau, label)
    if cfg_scale <= 0.0 or cfg_scale == 1.0:
        return eps_c, f_c[None]
    eps_u, f_u = forward(w, shape, x, tau, shape.n_classes)
    return eps_u + cfg_scale * (eps_c - eps_u), np.stack([f_c, f_u])


def verify_pass(w, shape, sched, x_states, t_idx, labels, cfg_scale: float):
    """The packed target pass (Alg. 1, parallel-means line; Sec. 3.3): every packed state is an
    independent sequence with its own schedule index and label.  Returns (means, eps, features)."""
    means, epss, feats = [], [], []
    for x, s, y in zip(x_states, t_idx, labels):
        eps, f = guided_eps(w, shape, x, sched.t_embed_value[int(s)], int(y), cfg_scale)
        means.append(sched.mean(x, eps, int(s)))
        epss.append(eps)
        feats.append(f)
    return np.stack(means), np.stack(epss), np.stack(feats)
