"""tcgen05 attention against the oracle's softmax(q k^T / sqrt(d)) v on bf16-representable inputs."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit as odit
from gpu_util import cu, nerr

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_seq,T,h,dh,gain", [(2, 256, 6, 64, 1.0), (1, 1024, 2, 72, 1.0), (3, 128, 1, 64, 1.0),
                                               (1, 256, 2, 96, 1.0), (1, 256, 1, 128, 1.0), (1, 384, 2, 40, 1.0),
                                               (2, 1024, 3, 72, 3.0), (5, 256, 16, 72, 0.3)])
def test_attention_tc(n_seq, T, h, dh, gain):
    from paper_2511_20390_b200 import binding as b
    qkv = synth.round_to_bf16(synth.normal(T + dh, 1, (n_seq, T, 3, h, dh), std=gain))
    got = b.op_attention(cu(qkv.reshape(n_seq, T, 3 * h * dh), torch.bfloat16), h)
    torch.cuda.synchronize()
    pick = [(0, 0), (n_seq - 1, h - 1), (n_seq // 2, h // 2)]
    for s, a in pick:
        ref = odit.attention(qkv[s, :, 0, a].astype(np.float64), qkv[s, :, 1, a].astype(np.float64), qkv[s, :, 2, a].astype(np.float64))
        e = nerr(got[s, :, a * dh:(a + 1) * dh], ref)
        assert e < 1e-2, (s, a, e)


def test_attention_peaked_rows():
    # one key dominates each row (large logits): the running-max rescaling must keep exactly that value
    from paper_2511_20390_b200 import binding as b
    T, h, dh = 256, 1, 64
    rng = np.random.default_rng(0)
    q = rng.standard_normal((T, dh)).astype(np.float32)
    k = q[rng.permutation(T)] * 6.0
    v = rng.standard_normal((T, dh)).astype(np.float32)
    qkv = synth.round_to_bf16(np.stack([q, k, v], axis=1)[None, :, :, None, :])
    got = b.op_attention(cu(qkv.reshape(1, T, 3 * dh), torch.bfloat16), h)
    ref = odit.attention(*(qkv[0, :, i, 0].astype(np.float64) for i in range(3)))
    assert nerr(got[0], ref) < 1e-2
