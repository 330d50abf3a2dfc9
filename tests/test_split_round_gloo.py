"""Bookkeeping of the packed pass partitioned over ranks (Sec. 4, wall-clock protocol: the drafts of a round verified on
parallel GPUs), on CPU with two gloo ranks: which rank owns which packed state, the in-place all-gather puts every
state's noise prediction at its packed position, and both ranks then take the same decisions, equal to those taken from
the unsplit tensor.  The predictions here are synthetic (no GPU); the decision rule is the oracle's."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_split_ranges_partition_the_packed_states():
    import paper_2511_20390_b200 as free
    from paper_2511_20390_b200.binding import FreeError
    for n, world in ((12, 1), (12, 2), (12, 3), (12, 4), (12, 6), (12, 12), (96, 8), (6, 6)):
        got = [free.split_range(n, world, r) for r in range(world)]
        assert got[0][0] == 0 and got[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(got, got[1:])) and len({hi - lo for lo, hi in got}) == 1
    # one image, as many GPUs as drafts: rank r verifies packed state r (one draft per GPU)
    assert [free.split_range(6, 6, r) for r in range(6)] == [(r, r + 1) for r in range(6)]
    for bad in ((12, 5, 0), (12, 2, 2), (12, 2, -1), (12, 0, 0)):
        with pytest.raises(FreeError) as e:
            free.split_range(*bad)
        assert e.value.code == -2


def _inputs():
    import synth
    B, K, G, shape = 3, 4, 2, (4, 8, 8)
    s2 = np.tile(np.array([0.02, 0.015, 0.01, 0.008], np.float32), (B, 1))
    sig = float(np.sqrt(s2.mean()))
    s = 0.35 * sig / np.sqrt(np.prod(shape))
    eps, x_first, mh, xh, u = synth.eps_verifier_inputs(77, B, K, G, shape, s, s2, eps_std=s / 0.05)
    cx, ce = np.ones((B, K), np.float32), np.full((B, K), 0.05, np.float32)
    return B, K, G, shape, eps, x_first, mh, xh, cx, ce, s2, u


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import paper_2511_20390_b200 as free
    from oracle import verify as ov
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, K, G, shape, eps, x_first, mh, xh, cx, ce, s2, u = _inputs()
    lo, hi = free.split_range(B * K, world, rank)
    full = torch.from_numpy(eps.reshape((B * K, G) + shape))
    eps_all = torch.full_like(full, float("nan"))
    eps_all[lo:hi] = full[lo:hi]                      # what this rank's share of the packed pass would have written
    try:
        dist.all_gather_into_tensor(eps_all, eps_all[lo:hi].clone())
    except (RuntimeError, NotImplementedError):       # a gloo build without the flat form: same exchange, list form
        parts = [torch.empty_like(eps_all[lo:hi]) for _ in range(world)]
        dist.all_gather(parts, eps_all[lo:hi].clone())
        eps_all = torch.cat(parts)
    in_order = bool(torch.equal(eps_all, full))       # gathered order = packed order, nothing left unfilled
    x, n, _, _ = ov.spec_verify_from_eps(eps_all.numpy().reshape((B, K, G) + shape), x_first, mh, xh, cx, ce, 4.0, s2, u)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, lo, hi, in_order, n.tolist(), float(np.abs(x).sum())))


def test_two_ranks_gather_in_packed_order_and_decide_alike():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31000 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, lo0, hi0, ok0, n0, x0), (r1, lo1, hi1, ok1, n1, x1) = res
    assert (lo0, hi0, lo1, hi1) == (0, 6, 6, 12) and ok0 and ok1
    assert n0 == n1 and x0 == x1                       # replicated decision: identical on both ranks
    # and equal to the decision taken from the unsplit tensor
    sys.path.insert(0, ROOT)
    from oracle import verify as ov
    B, K, G, shape, eps, x_first, mh, xh, cx, ce, s2, u = _inputs()
    x, n, _, _ = ov.spec_verify_from_eps(eps, x_first, mh, xh, cx, ce, 4.0, s2, u)
    assert n.tolist() == n0 and float(np.abs(x).sum()) == x0
    assert len(set(n0)) > 1                            # the samples do stop at different drafts
