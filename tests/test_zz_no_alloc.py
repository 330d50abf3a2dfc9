"""The allocation-free attention entry point (scratch built into the library's device image) must give what the
workspace-based entry point gives, on two calls in a row: the shared scratch keeps the first call's contents,
so the second call checks that nothing stale leaks through.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import synth

pytestmark = pytest.mark.gpu


def _qkv(seed, n_seq, T, h, dh):
    a = synth.round_to_bf16(synth.normal(seed, 1, (n_seq, T, 3 * h * dh)))
    return torch.from_numpy(a).to(torch.bfloat16).cuda()


def test_static_attention_matches_workspace_attention_twice():
    from paper_2511_20390_b200 import binding as b
    # first call: one DiT-XL/2-sized sequence (16 heads x 1024 tokens, d_head 72 padded to 80)
    q1 = _qkv(1, 1, 1024, 16, 72)
    ref1 = b.op_attention(q1, 16)
    got1 = b.op_attention_static(q1, 16)
    torch.cuda.synchronize()
    assert torch.isfinite(got1.float()).all()
    assert (got1.float() - ref1.float()).abs().max().item() <= 1e-2 * ref1.float().abs().max().item()
    # second call, different shape and padding (d_head 64, 3 sequences): reuses the same scratch bytes
    q2 = _qkv(2, 3, 256, 6, 64)
    ref2 = b.op_attention(q2, 6)
    got2 = b.op_attention_static(q2, 6)
    torch.cuda.synchronize()
    assert (got2.float() - ref2.float()).abs().max().item() <= 1e-2 * ref2.float().abs().max().item()
    # and the first problem again, after the scratch held the second one
    got3 = b.op_attention_static(q1, 16)
    assert torch.equal(got3, got1)


def test_static_attention_rejects_what_does_not_fit():
    from paper_2511_20390_b200 import binding as b
    too_big = _qkv(3, 2, 1024, 16, 72)          # 2 * 16 * 1024 * 80 elements > 2^21
    with pytest.raises(b.FreeError) as e:
        b.op_attention_static(too_big, 16)
    assert e.value.code == -6
    odd = _qkv(4, 1, 100, 2, 64)                # n_tok not a multiple of 128
    with pytest.raises(b.FreeError) as e:
        b.op_attention_static(odd, 2)
    assert e.value.code == -4
