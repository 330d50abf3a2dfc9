"""Helpers shared by the GPU parity tests: oracle-side batches and the error measure."""
import numpy as np
import torch


def cu(a, dt=torch.float32):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dt).cuda()


def nerr(got, ref):
    """max_i |got_i - ref_i| / max_i |ref_i| (elementwise relative error is undefined near zeros)."""
    got = got.detach().float().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    ref = np.asarray(ref, np.float64)
    return float(np.abs(got.astype(np.float64).reshape(ref.shape) - ref).max() / max(np.abs(ref).max(), 1e-30))
