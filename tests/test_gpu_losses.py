"""free_drafter_loss (CUDA, one fused reduction) against the oracle's objectives of Sec. 3.2 on identical inputs."""
import numpy as np
import pytest
import torch

import synth
from gpu_util import cu
from oracle import losses as olosses

pytestmark = pytest.mark.gpu


def _case(seed, n, n_tok, D, d_eps, bf16, spread=0.3):
    f_ref = synth.normal(seed, 1, (n, n_tok, D))
    f_pred = (f_ref + np.float32(spread) * synth.normal(seed, 2, (n, n_tok, D))).astype(np.float32)
    if bf16:
        f_ref, f_pred = synth.round_to_bf16(f_ref), synth.round_to_bf16(f_pred)
    e_ref = synth.normal(seed, 3, (n, d_eps))
    e_pred = (e_ref + np.float32(0.1) * synth.normal(seed, 4, (n, d_eps))).astype(np.float32)
    return e_pred, e_ref, f_pred, f_ref


@pytest.mark.parametrize("n,n_tok,D,d_eps,bf16", [
    (2, 256, 1152, 4096, True),        # DiT-XL/2 256^2 features
    (3, 64, 384, 1024, False),
    (1, 5, 7, 3, False),               # nothing divisible: scalar row loop, noise tail
    (2, 33, 24, 1030, True),           # rows of 24 (three 8-wide runs), noise tail of 2
    (40, 256, 1152, 4096, True),       # more rows than one pass of the grid
])
@pytest.mark.parametrize("beta", [1.0, 0.05])
def test_matches_oracle(n, n_tok, D, d_eps, bf16, beta):
    import paper_2511_20390_b200 as free
    e_pred, e_ref, f_pred, f_ref = _case(n + D, n, n_tok, D, d_eps, bf16)
    dt = torch.bfloat16 if bf16 else torch.float32
    out = free.drafter_loss(cu(e_pred), cu(e_ref), cu(f_pred, dt), cu(f_ref, dt), 0.5, 0.01, beta=beta, eps_cos=1e-8)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    ref = np.array(olosses.free_loss(e_pred, e_ref, f_pred, f_ref, 0.5, 0.01, beta=beta, eps_cos=1e-8))
    # rows are summed in fp32 lanes (D terms), everything beyond in fp64
    assert np.allclose(got, ref, rtol=2e-5, atol=1e-9), (got, ref)


def test_special_cases_and_determinism():
    import paper_2511_20390_b200 as free
    e_pred, e_ref, f_pred, f_ref = _case(5, 4, 128, 256, 2048, False)
    same = free.drafter_loss(cu(e_ref), cu(e_ref), cu(f_ref), cu(f_ref), 0.5, 0.01, eps_cos=0.0).cpu().numpy()
    assert same[0] == 0 and abs(same[1]) < 1e-6 and same[2] == 0
    flipped = free.drafter_loss(cu(e_ref), cu(e_ref), cu(-f_ref), cu(f_ref), 1.0, 0.0, eps_cos=0.0).cpu().numpy()
    assert abs(flipped[1] - 2.0) < 1e-6 and abs(flipped[3] - 2.0) < 1e-6
    a = free.drafter_loss(cu(e_pred), cu(e_ref), cu(f_pred), cu(f_ref), 0.5, 0.01).cpu().numpy()
    b = free.drafter_loss(cu(e_pred), cu(e_ref), cu(f_pred), cu(f_ref), 0.5, 0.01).cpu().numpy()
    assert np.array_equal(a, b)                                     # fixed reduction order: bit-identical repeats
    with pytest.raises(free.FreeError):
        free.drafter_loss(cu(e_pred), cu(e_ref), cu(f_pred), cu(f_ref), 0.5, 0.01, beta=0.0)
