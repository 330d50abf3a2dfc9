"""Feature-level autoregressive drafter in fp64 (TEST INFRASTRUCTURE ONLY).

Sec. 3.1: the drafter reuses the target's embedding layers, fuses the embedded
latent with the propagated top-block feature through one fully connected layer,
runs a single DiT block and a small output projection; the label embedding comes
from the target (Appendix "Training Details").  Where the paper is silent the
reading is: concatenation order [embedding, feature]; the FC layer has a bias and
no normalisation; the drafter is conditioned on the transition it predicts; it
has its own modulated output head; under guidance the conditional and the
unconditional streams each carry their own feature and the two noise predictions
are combined exactly as in the target.
"""
import numpy as np

from . import dit


def forward(w_t, w_d, shape, x_prev, f_prev, tau: float, label: int, n_blocks: int = 1):
    """(eps_hat [C,H,W], f_next [n_tok,D]) = p(. | x_prev, f_prev) for one sequence."""
    Wd = dit._with_heads(w_d, shape)
    sc = dit.silu(dit.conditioning(w_t, shape, tau, label))
    g = np.concatenate([dit.embed(w_t, shape, x_prev), np.asarray(f_prev, np.float64)], axis=1)
    h = dit.linear(g, w_d["fc_w"], w_d["fc_b"])
    for i in range(n_blocks):
        h = dit.block(h, sc, Wd, i)
    out = dit.final_layer(h, sc, Wd, shape)
    return out[:shape.C], h


def guided_step(w_t, w_d, shape, sched, x_prev, f_prev, s: int, label: int, cfg_scale: float, n_blocks: int = 1):
    """One drafter step for one state.  f_prev is [G, n_tok, D] (conditional first).  Returns
    (m_hat, eps_hat, f_next [G,n_tok,D]) for schedule index s."""
    tau = sched.t_embed_value[s]
    eps_c, f_c = forward(w_t, w_d, shape, x_prev, f_prev[0], tau, label, n_blocks)
    if cfg_scale <= 0.0 or cfg_scale == 1.0:
        eps, f = eps_c, f_c[None]
    else:
        eps_u, f_u = forward(w_t, w_d, shape, x_prev, f_prev[1], tau, shape.n_classes, n_blocks)
        eps, f = eps_u + cfg_scale * (eps_c - eps_u), np.stack([f_c, f_u])
    return sched.mean(x_prev, eps, s), eps, f
