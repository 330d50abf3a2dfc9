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
                                               (2, 1024, 3, 72, 3.0), (5, 256, 16, 72, 0.3),
                                               # more work items than SMs: persistent CTAs take several items each
                                               (10, 512, 16, 72, 1.0), (40, 256, 8, 64, 2.0), (3, 1024, 16, 72, 1.0)])
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


@pytest.mark.parametrize("T,h,dh,n_seq", [(1024, 2, 72, 1), (512, 1, 64, 1), (384, 1, 96, 1), (1024, 2, 72, 20)])
def test_attention_offset_moves_in_every_block(T, h, dh, n_seq):
    # logits along one direction grow from one block of 128 keys to the next by far more than the threshold at which
    # the exponent offset of a row is moved: rows with a positive projection rescale their accumulator in every block,
    # rows with a negative one keep the offset of their first block while later keys underflow to zero
    from paper_2511_20390_b200 import binding as b
    rng = np.random.default_rng(T + dh)
    e = rng.standard_normal(dh)
    e /= np.linalg.norm(e)
    sign = np.where(rng.random((T, 1)) < 0.5, -1.0, 1.0)
    qkv = np.zeros((1, T, 3, h, dh), np.float32)
    for a in range(h):
        q = sign * 3.0 * np.sqrt(dh) ** 0.5 * e + 0.3 * rng.standard_normal((T, dh))
        step = (np.arange(T) // 128 + 1.0)[:, None]                 # 1, 2, ... per block of keys
        k = step * 4.0 * np.sqrt(dh) ** 0.5 * e + 0.3 * rng.standard_normal((T, dh))
        qkv[0, :, 0, a], qkv[0, :, 1, a], qkv[0, :, 2, a] = q, k, rng.standard_normal((T, dh))
    qkv = synth.round_to_bf16(qkv)
    # n_seq > 1: the same sequence many times, so that persistent CTAs go through several work items each; the copies
    # must come out identical
    got = b.op_attention(cu(np.repeat(qkv, n_seq, axis=0).reshape(n_seq, T, 3 * h * dh), torch.bfloat16), h)
    torch.cuda.synchronize()
    for s_i in range(1, n_seq):
        assert torch.equal(got[s_i], got[0]), s_i
    for a in range(h):
        q64, k64, v64 = (qkv[0, :, i, a].astype(np.float64) for i in range(3))
        logits = q64 @ k64.T / np.sqrt(dh)
        rising = logits[:, -128:].max(1) - logits[:, :128].max(1)
        thr = 8.0 * (T // 128 - 1)                                  # ~11 per block of keys
        assert (rising > thr).sum() > T // 4 and (rising < -thr).sum() > T // 4   # both kinds of row are present
        ref = odit.attention(q64, k64, v64)
        assert np.isfinite(got[0, :, a * dh:(a + 1) * dh].float().cpu().numpy()).all()
        assert nerr(got[0, :, a * dh:(a + 1) * dh], ref) < 1e-2, a
