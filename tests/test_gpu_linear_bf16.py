"""tcgen05 linear layers (bf16 operands, fp32 accumulation) against the fp64 oracle on bf16-representable inputs."""
import numpy as np
import pytest
import torch

import synth
from oracle import dit as odit
from gpu_util import cu, nerr

pytestmark = pytest.mark.gpu


def _operands(M, N, K, seed):
    A = synth.round_to_bf16(synth.normal(seed, 1, (M, K)))
    W = synth.round_to_bf16(synth.normal(seed, 2, (N, K), std=0.05))
    bias = synth.normal(seed, 3, (N,))
    return A, W, bias


SHAPES = [(128, 32, 64), (128, 256, 64), (256, 192, 128), (300, 384, 192), (96, 64, 256), (1, 128, 64),
          (1000, 1152, 1152), (777, 3456, 384), (40000, 384, 64), (19500, 160, 128), (640, 4608, 1152), (512, 1152, 4608),
          (9000, 3456, 384), (6100, 4608, 128), (129, 192, 64), (300, 320, 128), (2049, 1152, 256),
          (700, 448, 128), (515, 704, 192), (260, 256, 64),        # last column block 192, 192 and none: every narrow width of the CTA-pair kernel
          # few row blocks: the CTA-pair kernel takes column blocks of 128 (one sequence, the two sequences of a batch-1
          # target step with the proj and fc2 shapes, a ragged last row block, two waves of narrow tiles)
          (1024, 1152, 1152), (2048, 1152, 1152), (2048, 1152, 4608), (1900, 1152, 1152), (4096, 1152, 1152), (2049, 1152, 1152)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_bias_fp32_out_is_exact_to_accumulation_order(M, N, K):
    from paper_2511_20390_b200 import binding as b
    A, W, bias = _operands(M, N, K, M + N + K)
    ref = odit.linear(A, W, bias)
    got = b.op_linear(cu(A, torch.bfloat16), cu(W, torch.bfloat16), cu(bias), out_dtype=b.FREE_FP32)
    # products of bf16 values are exact in fp32; only the fp32 accumulation order differs from fp64
    assert nerr(got, ref) < 2e-6 * max(1.0, np.sqrt(K / 64))


@pytest.mark.parametrize("M,N,K", [(300, 384, 192), (1000, 1152, 1152), (2048, 1152, 4608), (2048, 4608, 1152)])
def test_epilogues(M, N, K):
    from paper_2511_20390_b200 import binding as b
    A, W, bias = _operands(M, N, K, 5)
    ref = odit.linear(A, W, bias)
    a_, w_, b_ = cu(A, torch.bfloat16), cu(W, torch.bfloat16), cu(bias)
    assert nerr(b.op_linear(a_, w_, b_), ref) < 5e-3                                        # bf16 output rounding
    assert nerr(b.op_linear(a_, w_, b_, epilogue=b.EPI_BIAS_GELU, out_dtype=b.FREE_FP32), odit.gelu_tanh(ref)) < 1.5e-3   # tanh.approx
    assert nerr(b.op_linear(a_, w_, b_, epilogue=b.EPI_BIAS_GELU), odit.gelu_tanh(ref)) < 5e-3             # bf16 output
    assert nerr(b.op_linear(a_, w_, b_, epilogue=b.EPI_BIAS_SILU, out_dtype=b.FREE_FP32), odit.silu(ref)) < 1e-5
    assert nerr(b.op_linear(a_, w_, None, out_dtype=b.FREE_FP32), ref - bias) < 1e-5
    rps = 64
    nseq = (M + rps - 1) // rps
    gate, resid = synth.normal(6, 1, (nseq, 6 * N)), synth.normal(6, 2, (M, N))
    g = cu(gate)[:, 2 * N:3 * N]
    out = b.op_linear(a_, w_, b_, epilogue=b.EPI_GATE_RESIDUAL, resid=cu(resid), gate=g, rows_per_seq=rps)
    ref_r = resid + np.repeat(gate[:, 2 * N:3 * N], rps, axis=0)[:M] * ref
    assert nerr(out, ref_r) < 1e-5
    out = b.op_linear(a_, w_, None, epilogue=b.EPI_GATE_RESIDUAL, resid=cu(resid), gate=None)
    assert nerr(out, resid + ref - bias) < 1e-5


def test_repeated_calls_are_deterministic():
    from paper_2511_20390_b200 import binding as b
    A, W, bias = _operands(5000, 1152, 1152, 9)
    a_, w_, b_ = cu(A, torch.bfloat16), cu(W, torch.bfloat16), cu(bias)
    first = b.op_linear(a_, w_, b_, out_dtype=b.FREE_FP32).clone()
    for _ in range(3):
        assert torch.equal(first, b.op_linear(a_, w_, b_, out_dtype=b.FREE_FP32))


def test_unsupported_shapes_are_refused():
    from paper_2511_20390_b200 import binding as b
    A, W, bias = _operands(64, 48, 64, 1)          # N not a multiple of 32
    with pytest.raises(b.FreeError) as e:
        b.op_linear(cu(A, torch.bfloat16), cu(W, torch.bfloat16), cu(bias))
    assert e.value.code == -4
