"""A round with its packed target pass partitioned over ranks (free_spec_round_begin / free_spec_round_finish) against the
one-call round on the same inputs, on ONE GPU: the ranks' shares are computed one after the other into the same tensor of
noise predictions (what the all-gather produces on every rank), then the replicated second half runs once.  Nothing here
waits on another launch; the exchange itself is covered on CPU (tests/test_split_round_gloo.py)."""
import dataclasses

import numpy as np
import pytest
import torch

import synth
from gpu_util import cu

pytestmark = pytest.mark.gpu


def _setup(free, sh, B, N, bf16):
    shape = (sh.C, sh.H, sh.W)
    w = synth.make_target_weights(sh, 31, bf16=bf16, ada_std=0.2, out_gain=2.0)
    wd = synth.make_drafter_weights(sh, 32, bf16=bf16, ada_std=0.2, out_gain=2.0)
    model = free.Model(sh, w, wd, dtype="bf16" if bf16 else "fp32")
    dsched = free.DeviceSchedule(free.respaced_schedule(N) if N == 250 else free.linear_schedule(N))
    x0 = cu(synth.normal(6, 1, (B,) + shape))
    zt, zd = cu(synth.normal(6, 2, (B, N) + shape)), cu(synth.normal(6, 3, (B, N) + shape))
    uu = synth.uniform01(6, 4, (B, N))
    uu[uu < 0.7] = 0.0                                 # u = 0 always accepts: the samples stop at different drafts
    u = cu(uu)
    return model, dsched, x0, zt, zd, u


@pytest.mark.parametrize("world", [1, 2, 3, 4, 6, 12])
def test_partitioned_round_equals_the_one_call_round_s2(world):
    import paper_2511_20390_b200 as free
    sh = dataclasses.replace(synth.DIT_S2, depth=3)
    B, K, N, cfg = 2, 6, 250, 4.0
    model, dsched, x0, zt, zd, u = _setup(free, sh, B, N, True)
    labels = cu(np.array([5, 800], np.int32), torch.int32)
    cursor = cu(np.array([30, 244], np.int32), torch.int32)      # the second sample has 5 drafts left, not 6
    ref = [t.clone() for t in model.spec_round(x0, cursor, labels, dsched, K, cfg, zt, zd, u)]
    eps_all = torch.full((B * K, 2, sh.C, sh.H, sh.W), float("nan"), device="cuda")
    covered = torch.zeros(B * K, dtype=torch.bool)
    for rank in range(world):                                     # each rank's begin fills its own slice only
        before = eps_all.clone()
        _, lo, hi = model.spec_round_begin(x0, cursor, labels, dsched, K, cfg, zt, zd, u, rank, world, eps_all=eps_all)
        torch.cuda.synchronize()
        changed = (~((eps_all == before) | (eps_all.isnan() & before.isnan()))).flatten(1).any(1).cpu()
        assert changed[lo:hi].all() and not changed[:lo].any() and not changed[hi:].any()
        covered[lo:hi] = True
    assert covered.all() and torch.isfinite(eps_all).all()
    got = model.spec_round_finish(eps_all, labels, dsched, K, cfg, zt, zd, u, x0)
    torch.cuda.synchronize()
    assert model.device_error() == 0
    assert torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2]) and torch.equal(got[0], ref[0])
    assert ref[1].tolist()[1] <= N + 1 and 0 < sum(ref[2].tolist()) <= 2 * K


def test_partitioned_round_tiny_fp32_and_argument_errors():
    import paper_2511_20390_b200 as free
    from paper_2511_20390_b200.binding import FreeError
    sh = synth.TINY
    B, K, N = 2, 6, 50
    model, dsched, x0, zt, zd, u = _setup(free, sh, B, N, False)
    labels = cu(np.array([1, 9], np.int32), torch.int32)
    cursor = cu(np.array([3, 20], np.int32), torch.int32)
    ref = [t.clone() for t in model.spec_round(x0, cursor, labels, dsched, K, 0.0, zt, zd, u)]
    eps_all = None
    for rank in range(4):
        eps_all, lo, hi = model.spec_round_begin(x0, cursor, labels, dsched, K, 0.0, zt, zd, u, rank, 4, eps_all=eps_all)
        assert (lo, hi) == (3 * rank, 3 * rank + 3)
    got = model.spec_round_finish(eps_all, labels, dsched, K, 0.0, zt, zd, u, x0)
    assert all(torch.equal(a, b) for a, b in zip(got, ref))
    # world == 1 through the composed call (no exchange needed)
    got1 = model.spec_round_split(x0, cursor, labels, dsched, K, 0.0, zt, zd, u, 0, 1)
    assert all(torch.equal(a, b) for a, b in zip(got1, ref))
    with pytest.raises(FreeError) as e:                            # 12 packed states do not divide over 5 ranks
        model.spec_round_begin(x0, cursor, labels, dsched, K, 0.0, zt, zd, u, 0, 5)
    assert e.value.code == -2
