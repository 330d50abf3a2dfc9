"""ctypes binding of libfree_b200.so: argument marshalling only.

Tensors are torch CUDA tensors (device memory owner); the library receives raw device pointers and
the current stream.  Nothing here computes any part of the method.
"""
import ctypes as C
import os

import numpy as np
import torch

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libfree_b200.so")

FREE_FP32, FREE_BF16 = 0, 1
FREE_MAX_K = 64
EPI_BIAS, EPI_BIAS_GELU, EPI_BIAS_SILU, EPI_GATE_RESIDUAL = 0, 1, 2, 3


class FreeError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: error {code} ({lib().free_strerror(code).decode()})")


class BlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ada_w", "ada_b", "qkv_w", "qkv_b", "proj_w", "proj_b",
                                          "fc1_w", "fc1_b", "fc2_w", "fc2_b")]


class ModelDesc(C.Structure):
    _fields_ = ([(n, C.c_int32) for n in ("dtype", "C", "H", "W", "patch", "D", "depth", "heads",
                                          "n_classes", "c_out", "freq_dim", "mlp_ratio")]
                + [(n, C.c_void_p) for n in ("t_w1", "t_b1", "t_w2", "t_b2", "y_emb", "pe_w", "pe_b", "pos")]
                + [("blocks", BlockWeights)]
                + [(n, C.c_void_p) for n in ("fada_w", "fada_b", "fin_w", "fin_b")])


class DrafterDesc(C.Structure):
    _fields_ = ([("n_blocks", C.c_int32)] + [(n, C.c_void_p) for n in ("fc_w", "fc_b")]
                + [("blocks", BlockWeights)]
                + [(n, C.c_void_p) for n in ("fada_w", "fada_b", "fin_w", "fin_b")])


class ScheduleDesc(C.Structure):
    _fields_ = [("N", C.c_int32)] + [(n, C.c_void_p) for n in ("coef_x", "coef_eps", "sigma2", "t_embed_value")]


class SpecParams(C.Structure):
    _fields_ = [("K", C.c_int32), ("cfg_scale", C.c_float), ("lam", C.c_void_p)]


class TrajStats(C.Structure):
    _fields_ = [("rounds", C.c_int64), ("target_calls", C.c_int64), ("draft_calls", C.c_int64),
                ("accepted", C.c_int64), ("rejected", C.c_int64),
                ("accept_hist", C.c_int64 * (FREE_MAX_K + 1)), ("parallel_efficiency", C.c_double)]


_LIB = None

_SIGNATURES = {
    "free_strerror": (C.c_char_p, [C.c_int]),
    "free_create": (C.c_int, [C.POINTER(ModelDesc), C.POINTER(DrafterDesc), C.POINTER(C.c_void_p)]),
    "free_destroy": (C.c_int, [C.c_void_p]),
    "free_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int]),
    "dit_verify_pass": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                  C.POINTER(ScheduleDesc), C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_void_p]),
    "spec_verify": (C.c_int, [C.c_int, C.c_int, C.c_int64] + [C.c_void_p] * 11),
    "draft_step": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                             C.POINTER(ScheduleDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_size_t, C.c_void_p]),
    "sample_trajectory": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.POINTER(ScheduleDesc),
                                    C.POINTER(SpecParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.POINTER(TrajStats), C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_op_linear_workspace_bytes": (C.c_size_t, []),
    "free_op_linear": (C.c_int, [C.c_int] * 6 + [C.c_void_p] * 6 + [C.c_int64, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_op_ln_modulate": (C.c_int, [C.c_int] * 4 + [C.c_void_p] * 3 + [C.c_int64, C.c_void_p, C.c_void_p]),
    "free_op_attention": (C.c_int, [C.c_int] * 5 + [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_op_attention_workspace_bytes": (C.c_size_t, [C.c_int] * 5),
}


def exported_symbols():
    return sorted(_SIGNATURES)


def lib():
    """The loaded shared library; raises if it has not been built (there is no fallback path)."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_20390_b200.build`")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)          # AttributeError if the library does not export it
            fn.restype, fn.argtypes = res, args
        _LIB = L
    return _LIB


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code, what):
    if code != 0:
        raise FreeError(code, what)


def _dev(t, dtype):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise ValueError("expected a contiguous CUDA tensor of dtype %s" % dtype)
    return t


# ------------------------------------------------------------------------------------------ verifier
def spec_verify(m, m_hat, x_hat, sigma2, u, lam=None, n_valid=None, want_logratio=False,
                x_out=None, n_accept=None):
    """Algorithm 2 over K drafts per sample with the first-rejection break (strict, or relaxed when
    `lam` is given).  m, m_hat, x_hat: CUDA fp32 [B,K,d...]; sigma2, u, lam: [B,K]; n_valid int32 [B].
    Returns (x_out [B,d...], n_accept int32 [B][, ell [B,K]])."""
    B, K = m.shape[:2]
    d = int(np.prod(m.shape[2:]))
    for t in (m, m_hat, x_hat, sigma2, u):
        _dev(t, torch.float32)
    if x_out is None:
        x_out = torch.zeros((B,) + tuple(m.shape[2:]), dtype=torch.float32, device=m.device)
    if n_accept is None:
        n_accept = torch.empty(B, dtype=torch.int32, device=m.device)
    ell = torch.empty((B, K), dtype=torch.float32, device=m.device) if want_logratio else None
    code = lib().spec_verify(B, K, d, _ptr(m), _ptr(m_hat), _ptr(x_hat), _ptr(sigma2),
                             _ptr(None if lam is None else _dev(lam, torch.float32)), _ptr(u),
                             _ptr(None if n_valid is None else _dev(n_valid, torch.int32)),
                             _ptr(x_out), _ptr(n_accept), _ptr(ell), _stream())
    _check(code, "spec_verify")
    return (x_out, n_accept, ell) if want_logratio else (x_out, n_accept)


class HostVerifier:
    """spec_verify on HOST buffers: pinned staging, host->device copies, the kernel, device->host copies
    of the result, all on the current stream (the end-to-end path of the benchmark)."""

    def __init__(self, B, K, d, relaxed=False):
        self.shape = (B, K, d)
        pin = lambda *s, dt=torch.float32: torch.empty(*s, dtype=dt, pin_memory=True)
        dev = lambda *s, dt=torch.float32: torch.empty(*s, dtype=dt, device="cuda")
        self.h = {n: pin(B, K, d) for n in ("m", "m_hat", "x_hat")}
        self.h.update({n: pin(B, K) for n in ("sigma2", "u")})
        if relaxed:
            self.h["lam"] = pin(B, K)
        self.d = {n: dev(*t.shape) for n, t in self.h.items()}
        self.x_out, self.n_accept = dev(B, d), dev(B, dt=torch.int32)
        self.h_x_out, self.h_n_accept = pin(B, d), pin(B, dt=torch.int32)
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in self.h.values())
        self.d2h_bytes = self.h_x_out.numel() * 4 + self.h_n_accept.numel() * 4

    def load(self, **arrays):
        for n, a in arrays.items():
            self.h[n].copy_(torch.from_numpy(np.ascontiguousarray(a)).reshape(self.h[n].shape))

    def run(self):
        for n, t in self.h.items():
            self.d[n].copy_(t, non_blocking=True)
        spec_verify(self.d["m"], self.d["m_hat"], self.d["x_hat"], self.d["sigma2"], self.d["u"],
                    lam=self.d.get("lam"), x_out=self.x_out, n_accept=self.n_accept)
        self.h_x_out.copy_(self.x_out, non_blocking=True)
        self.h_n_accept.copy_(self.n_accept, non_blocking=True)
        return self.h_x_out, self.h_n_accept


def spec_verify_host(m, m_hat, x_hat, sigma2, u, lam=None):
    """Convenience wrapper: numpy in, numpy out, through HostVerifier."""
    B, K = m.shape[:2]
    d = int(np.prod(m.shape[2:]))
    hv = HostVerifier(B, K, d, relaxed=lam is not None)
    args = dict(m=m, m_hat=m_hat, x_hat=x_hat, sigma2=sigma2, u=u)
    if lam is not None:
        args["lam"] = lam
    hv.load(**args)
    x, n = hv.run()
    torch.cuda.current_stream().synchronize()
    return x.numpy().reshape((B,) + tuple(m.shape[2:])).copy(), n.numpy().copy()
