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
    _fields_ = [("K", C.c_int32), ("cfg_scale", C.c_float), ("lam", C.c_void_p), ("use_graph", C.c_int32)]


class ProfEntry(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int64), ("ms", C.c_double), ("work", C.c_double)]


class TrajStats(C.Structure):
    _fields_ = [("rounds", C.c_int64), ("target_calls", C.c_int64), ("draft_calls", C.c_int64),
                ("accepted", C.c_int64), ("rejected", C.c_int64),
                ("accept_hist", C.c_int64 * (FREE_MAX_K + 1)), ("parallel_efficiency", C.c_double),
                ("graph_rounds", C.c_int64)]


_LIB = None

_SIGNATURES = {
    "free_strerror": (C.c_char_p, [C.c_int]),
    "free_create": (C.c_int, [C.POINTER(ModelDesc), C.POINTER(DrafterDesc), C.POINTER(C.c_void_p)]),
    "free_destroy": (C.c_int, [C.c_void_p]),
    "free_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int]),
    "dit_verify_pass": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                  C.POINTER(ScheduleDesc), C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_void_p]),
    "dit_verify_pass_raw": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                      C.POINTER(ScheduleDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "spec_verify": (C.c_int, [C.c_int, C.c_int, C.c_int64] + [C.c_void_p] * 11),
    "spec_verify_fused": (C.c_int, [C.c_int, C.c_int, C.c_int64, C.c_int, C.c_float] + [C.c_void_p] * 10 + [C.c_int] + [C.c_void_p] * 6),
    "draft_step": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                             C.POINTER(ScheduleDesc), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                             C.c_void_p, C.c_size_t, C.c_void_p]),
    "sample_trajectory": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.POINTER(ScheduleDesc),
                                    C.POINTER(SpecParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                    C.POINTER(TrajStats), C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_spec_round": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ScheduleDesc),
                                  C.POINTER(SpecParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_split_range": (C.c_int, [C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "free_spec_round_begin": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ScheduleDesc),
                                        C.POINTER(SpecParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_spec_round_finish": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.POINTER(ScheduleDesc), C.POINTER(SpecParams),
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_uncertainty_profile": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.POINTER(ScheduleDesc),
                                           C.POINTER(SpecParams), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_schedule_linear": (C.c_int, [C.c_int, C.c_double, C.c_double, C.c_int, C.c_double, C.c_double] + [C.c_void_p] * 4),
    "free_schedule_respaced": (C.c_int, [C.c_int, C.c_int, C.c_double, C.c_double, C.c_int, C.c_double, C.c_double] + [C.c_void_p] * 4),
    "free_fit_lambda_profile": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "free_drafter_loss_workspace_bytes": (C.c_size_t, []),
    "free_drafter_loss": (C.c_int, [C.c_int] * 4 + [C.c_int64] + [C.c_void_p] * 4 + [C.c_float] * 4 +
                          [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_set_launch_overlap": (C.c_int, [C.c_int]),
    "free_device_error_code": (C.c_int, [C.c_uint32]),
    "free_selftest_bounded_wait": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]),
    "free_profile_begin": (C.c_int, [C.c_void_p]),
    "free_profile_end": (C.c_int, [C.c_void_p, C.POINTER(ProfEntry), C.c_int, C.POINTER(C.c_int)]),
    "free_op_linear_workspace_bytes": (C.c_size_t, []),
    "free_op_linear": (C.c_int, [C.c_int] * 6 + [C.c_void_p] * 6 + [C.c_int64, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_op_ln_modulate": (C.c_int, [C.c_int] * 4 + [C.c_void_p] * 3 + [C.c_int64, C.c_void_p, C.c_void_p]),
    "free_op_attention": (C.c_int, [C.c_int] * 5 + [C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "free_op_attention_workspace_bytes": (C.c_size_t, [C.c_int] * 5),
    "free_op_attention_static": (C.c_int, [C.c_int] * 4 + [C.c_void_p] * 4),
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


def spec_verify_fused(eps, x_first, m_hat, x_hat, coef_x, coef_eps, sigma2, u, cfg_scale, lam=None,
                      n_valid=None, chunk=0, want_logratio=False, want_means=False, want_dist2=False, x_out=None, n_accept=None):
    """Verification straight from the packed pass's noise predictions (guidance, Eq. ddpm_update and Algorithm 2 in
    one kernel).  eps: CUDA fp32 [B,K,G,d...]; x_first [B,d...]; m_hat, x_hat [B,K,d...]; coef_x, coef_eps, sigma2, u,
    lam: [B,K]; chunk > 0 enables the early exit.  Returns (x_out, n_accept[, ell][, means][, dist2])."""
    B, K, G = eps.shape[:3]
    d = int(np.prod(eps.shape[3:]))
    for t in (eps, x_first, m_hat, x_hat, coef_x, coef_eps, sigma2, u):
        _dev(t, torch.float32)
    dev = eps.device
    if x_out is None:
        x_out = torch.zeros((B,) + tuple(eps.shape[3:]), dtype=torch.float32, device=dev)
    if n_accept is None:
        n_accept = torch.empty(B, dtype=torch.int32, device=dev)
    ell = torch.empty((B, K), dtype=torch.float32, device=dev) if want_logratio else None
    means = torch.zeros((B, K) + tuple(eps.shape[3:]), dtype=torch.float32, device=dev) if want_means else None
    dist2 = torch.empty((B, K), dtype=torch.float32, device=dev) if want_dist2 else None
    code = lib().spec_verify_fused(B, K, d, G, float(cfg_scale), _ptr(eps), _ptr(x_first),
                                   _ptr(m_hat), _ptr(x_hat), _ptr(coef_x), _ptr(coef_eps), _ptr(sigma2),
                                   _ptr(None if lam is None else _dev(lam, torch.float32)), _ptr(u),
                                   _ptr(None if n_valid is None else _dev(n_valid, torch.int32)), int(chunk),
                                   _ptr(x_out), _ptr(n_accept), _ptr(ell), _ptr(dist2), _ptr(means), _stream())
    _check(code, "spec_verify_fused")
    return ((x_out, n_accept) + ((ell,) if want_logratio else ()) + ((means,) if want_means else ())
            + ((dist2,) if want_dist2 else ()))


_LOSS_WS = {}


def drafter_loss(eps_pred, eps_ref, f_pred, f_ref, lambda_f, lambda_s, beta=1.0, eps_cos=1e-8, out=None):
    """Drafter training objectives (Sec. 3.2) in one fused reduction.  eps_*: CUDA fp32 [n, d...]; f_*: CUDA fp32 or
    bf16 [n, n_tok, D].  Returns a CUDA float64 tensor (L_noise, L_feat, L_smooth, L_total)."""
    n, n_tok, D = f_pred.shape
    _dev(eps_pred, torch.float32); _dev(eps_ref, torch.float32); _dev(f_ref, f_pred.dtype)
    dtype = {torch.float32: FREE_FP32, torch.bfloat16: FREE_BF16}[f_pred.dtype]
    _dev(f_pred, f_pred.dtype)
    if out is None:
        out = torch.empty(4, dtype=torch.float64, device=f_pred.device)
    ws = _LOSS_WS.get(f_pred.device)
    if ws is None:
        ws = _LOSS_WS[f_pred.device] = torch.empty(lib().free_drafter_loss_workspace_bytes(), dtype=torch.uint8, device=f_pred.device)
    _check(lib().free_drafter_loss(dtype, n, n_tok, D, eps_pred.numel() // n, _ptr(eps_pred), _ptr(eps_ref), _ptr(f_pred), _ptr(f_ref),
                                   float(lambda_f), float(lambda_s), float(beta), float(eps_cos), _ptr(out), _ptr(ws), ws.numel(),
                                   _stream()), "free_drafter_loss")
    return out


def fit_lambda_profile(eps_delta, count=None, window=0):
    """Relaxation table (Sec. 3.4) from per-transition prediction deviations: host-side fit inside the library.
    eps_delta: [N] (index n-1 for transition n); count: [N] measurements per transition or None.  Returns fp32 [N]."""
    e = np.ascontiguousarray(eps_delta, dtype=np.float64)
    c = None if count is None else np.ascontiguousarray(count, dtype=np.int64)
    out = np.empty(len(e), dtype=np.float32)
    code = lib().free_fit_lambda_profile(e.ctypes.data_as(C.c_void_p), None if c is None else c.ctypes.data_as(C.c_void_p),
                                         len(e), int(window), out.ctypes.data_as(C.c_void_p))
    _check(code, "free_fit_lambda_profile")
    return out


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


# ------------------------------------------------------------------------------------------ model
_ACT = {FREE_FP32: torch.float32, FREE_BF16: torch.bfloat16}
_MATRICES = ("t_w1", "t_w2", "ada_w", "qkv_w", "proj_w", "fc1_w", "fc2_w", "fada_w", "fc_w")


def split_range(n_states: int, world: int, rank: int):
    """The packed states [lo, hi) that `rank` of `world` owns (free_split_range)."""
    lo, hi = C.c_int(0), C.c_int(0)
    _check(lib().free_split_range(int(n_states), int(world), int(rank), C.byref(lo), C.byref(hi)), "free_split_range")
    return lo.value, hi.value


def selftest_bounded_wait(limit_cycles: int = 100_000):
    """Runs the pipelines' bounded wait once on a barrier nothing signals (free_selftest_bounded_wait).  Returns
    (error word, SM cycles waited, library return code the word maps to)."""
    err = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(lib().free_selftest_bounded_wait(_ptr(err), int(limit_cycles), _ptr(waited), _stream()), "free_selftest_bounded_wait")
    torch.cuda.current_stream().synchronize()
    word = int(err.item()) & 0xFFFFFFFF
    return word, int(waited.item()), int(lib().free_device_error_code(word))


class DeviceSchedule:
    """The four reverse-process tables (see paper_2511_20390_b200.schedule) as fp32 device arrays."""

    def __init__(self, tables: dict, device="cuda"):
        self.N = int(len(tables["sigma2"]))
        self.t = {k: torch.tensor(np.asarray(v, dtype=np.float32), device=device) for k, v in tables.items()}
        self.desc = ScheduleDesc(self.N, *(self.t[k].data_ptr() for k in ("coef_x", "coef_eps", "sigma2", "t_embed_value")))


def _upload(weights: dict, dtype: int, device):
    out = {}
    for k, v in weights.items():
        if isinstance(v, torch.Tensor):
            t = v.to(device)
            out[k] = (t.to(_ACT[dtype]) if k in _MATRICES else t.to(torch.float32)).contiguous()
            continue
        t = torch.from_numpy(np.ascontiguousarray(v, dtype=np.float32)).to(device)
        out[k] = t.to(_ACT[dtype]).contiguous() if k in _MATRICES else t
    return out


def _block_desc(w):
    return BlockWeights(*(w[k].data_ptr() for k in ("ada_w", "ada_b", "qkv_w", "qkv_b", "proj_w", "proj_b",
                                                    "fc1_w", "fc1_b", "fc2_w", "fc2_b")))


class Model:
    """A target DiT (and optionally a drafter) resident on the GPU, bound to a library context.

    `shape` carries the dimensions (fields C, H, W, patch, D, depth, heads, n_classes, c_out, freq_dim,
    mlp_ratio); `weights` / `drafter_weights` are dicts of host arrays laid out as the public header
    describes.  dtype "fp32" or "bf16" selects the compute mode.
    """

    def __init__(self, shape, weights: dict, drafter_weights: dict | None = None, dtype: str = "bf16",
                 n_draft_blocks: int = 1, device="cuda"):
        self.shape, self.dtype = shape, {"fp32": FREE_FP32, "bf16": FREE_BF16}[dtype]
        self.act = _ACT[self.dtype]
        self.device = torch.device(device)
        self.w = _upload(weights, self.dtype, self.device)
        w = self.w
        md = ModelDesc(self.dtype, shape.C, shape.H, shape.W, shape.patch, shape.D, shape.depth, shape.heads,
                       shape.n_classes, shape.c_out, shape.freq_dim, shape.mlp_ratio,
                       *(w[k].data_ptr() for k in ("t_w1", "t_b1", "t_w2", "t_b2", "y_emb", "pe_w", "pe_b", "pos")),
                       _block_desc(w), *(w[k].data_ptr() for k in ("fada_w", "fada_b", "fin_w", "fin_b")))
        dd = None
        self.wd = None
        if drafter_weights is not None:
            self.wd = _upload(drafter_weights, self.dtype, self.device)
            wd = self.wd
            dd = DrafterDesc(n_draft_blocks, wd["fc_w"].data_ptr(), wd["fc_b"].data_ptr(), _block_desc(wd),
                             *(wd[k].data_ptr() for k in ("fada_w", "fada_b", "fin_w", "fin_b")))
        self.ctx = C.c_void_p()
        _check(lib().free_create(C.byref(md), C.byref(dd) if dd is not None else None, C.byref(self.ctx)), "free_create")
        self._ws = None

    def __del__(self):
        try:
            if getattr(self, "ctx", None):
                lib().free_destroy(self.ctx)
                self.ctx = None
        except Exception:
            pass

    def workspace(self, n_states: int):
        need = lib().free_workspace_bytes(self.ctx, int(n_states))
        if self._ws is None or self._ws.numel() < need:
            self._ws = None
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    @classmethod
    def random(cls, shape, seed: int, dtype: str = "bf16", with_drafter: bool = True, n_draft_blocks: int = 1,
               std: float = 0.02, device="cuda"):
        """Random-init model whose weights are drawn on the device (no host copy): for timing runs, where the
        values only need the right shapes and scale.  The fixed position table comes from `synth`."""
        import synth
        g = torch.Generator(device=device)
        g.manual_seed(int(seed))
        D, F = shape.D, shape.mlp_ratio * shape.D
        act = _ACT[{"fp32": FREE_FP32, "bf16": FREE_BF16}[dtype]]

        def mat(*s):
            return (torch.randn(*s, generator=g, device=device, dtype=torch.float32) * std).to(act)

        def vec(*s):
            return torch.randn(*s, generator=g, device=device, dtype=torch.float32) * std

        def blocks(n):
            return {"ada_w": mat(n, 6 * D, D), "ada_b": vec(n, 6 * D), "qkv_w": mat(n, 3 * D, D), "qkv_b": vec(n, 3 * D),
                    "proj_w": mat(n, D, D), "proj_b": vec(n, D), "fc1_w": mat(n, F, D), "fc1_b": vec(n, F),
                    "fc2_w": mat(n, D, F), "fc2_b": vec(n, D), "fada_w": mat(2 * D, D), "fada_b": vec(2 * D),
                    "fin_w": vec(shape.out_dim, D), "fin_b": vec(shape.out_dim)}
        w = {"t_w1": mat(D, shape.freq_dim), "t_b1": vec(D), "t_w2": mat(D, D), "t_b2": vec(D),
             "y_emb": vec(shape.n_classes + 1, D), "pe_w": vec(D, shape.patch_dim), "pe_b": vec(D),
             "pos": torch.from_numpy(synth.pos_embed_2d(shape)).to(device)}
        w.update(blocks(shape.depth))
        wd = None
        if with_drafter:
            wd = {"fc_w": mat(D, 2 * D), "fc_b": vec(D)}
            wd.update(blocks(n_draft_blocks))
        return cls(shape, w, wd, dtype=dtype, n_draft_blocks=n_draft_blocks, device=device)

    def device_error(self) -> int:
        """The device error word of the last call that used the workspace (0 = no bounded wait gave up).
        Synchronises the current stream."""
        if self._ws is None:
            return 0
        torch.cuda.current_stream().synchronize()
        return int(self._ws[:4].view(torch.int32).item())

    def profile_begin(self):
        _check(lib().free_profile_begin(self.ctx), "free_profile_begin")

    def profile_end(self):
        """Per-kernel-class totals since profile_begin(): list of dicts name / launches / ms / work."""
        buf = (ProfEntry * 32)()
        n = C.c_int(0)
        _check(lib().free_profile_end(self.ctx, buf, 32, C.byref(n)), "free_profile_end")
        return [{"name": buf[i].name.decode(), "launches": buf[i].launches, "ms": buf[i].ms, "work": buf[i].work}
                for i in range(n.value)]

    def spec_round(self, x_cur, cursor, labels, sched, K, cfg_scale, noise_target, noise_draft=None, uniforms=None,
                   lam=None, x_next=None, cursor_next=None, n_accept=None):
        """One round of Algorithm 1 (asynchronous).  Returns (x_next, cursor_next, n_accept)."""
        B = x_cur.shape[0]
        _dev(x_cur, torch.float32); _dev(cursor, torch.int32); _dev(labels, torch.int32)
        prm = SpecParams(int(K), float(cfg_scale), None if lam is None else _dev(lam, torch.float32).data_ptr())
        x_next = torch.empty_like(x_cur) if x_next is None else x_next
        cursor_next = torch.empty_like(cursor) if cursor_next is None else cursor_next
        n_accept = torch.zeros(B, dtype=torch.int32, device=x_cur.device) if n_accept is None else n_accept
        ws = self.workspace(B * max(int(K), 1))
        _check(lib().free_spec_round(self.ctx, B, _ptr(x_cur), _ptr(cursor), _ptr(labels), C.byref(sched.desc), C.byref(prm),
                                     _ptr(noise_target), _ptr(noise_draft), _ptr(uniforms), _ptr(x_next), _ptr(cursor_next),
                                     _ptr(n_accept), _ptr(ws), ws.numel(), _stream()), "free_spec_round")
        return x_next, cursor_next, n_accept

    def spec_round_begin(self, x_cur, cursor, labels, sched, K, cfg_scale, noise_target, noise_draft, uniforms, rank, world,
                         eps_all=None, lam=None):
        """First half of a round whose packed pass is partitioned over `world` ranks (free_spec_round_begin): target step,
        drafter steps, and the packed pass over this rank's states, written into eps_all [B*K, G, C, H, W] in place.
        Returns (eps_all, lo, hi)."""
        B, sh = x_cur.shape[0], self.shape
        _dev(x_cur, torch.float32); _dev(cursor, torch.int32); _dev(labels, torch.int32)
        prm = SpecParams(int(K), float(cfg_scale), None if lam is None else _dev(lam, torch.float32).data_ptr())
        lo, hi = split_range(B * int(K), world, rank)
        if eps_all is None:
            eps_all = torch.empty((B * int(K), self.guided(cfg_scale), sh.C, sh.H, sh.W), dtype=torch.float32, device=x_cur.device)
        ws = self.workspace(B * int(K))
        _check(lib().free_spec_round_begin(self.ctx, B, _ptr(x_cur), _ptr(cursor), _ptr(labels), C.byref(sched.desc), C.byref(prm),
                                           _ptr(noise_target), _ptr(noise_draft), _ptr(uniforms), int(rank), int(world), _ptr(eps_all),
                                           _ptr(ws), ws.numel(), _stream()), "free_spec_round_begin")
        return eps_all, lo, hi

    def spec_round_finish(self, eps_all, labels, sched, K, cfg_scale, noise_target, noise_draft, uniforms, like, lam=None,
                          x_next=None, cursor_next=None, n_accept=None):
        """Second half (free_spec_round_finish): verification and cursor update on the gathered predictions.  `like` is the
        round's x_cur (shape and device of the outputs).  Returns (x_next, cursor_next, n_accept)."""
        B = like.shape[0]
        prm = SpecParams(int(K), float(cfg_scale), None if lam is None else _dev(lam, torch.float32).data_ptr())
        x_next = torch.empty_like(like) if x_next is None else x_next
        cursor_next = torch.empty(B, dtype=torch.int32, device=like.device) if cursor_next is None else cursor_next
        n_accept = torch.zeros(B, dtype=torch.int32, device=like.device) if n_accept is None else n_accept
        ws = self.workspace(B * int(K))
        _check(lib().free_spec_round_finish(self.ctx, B, _ptr(labels), C.byref(sched.desc), C.byref(prm), _ptr(noise_target),
                                            _ptr(noise_draft), _ptr(uniforms), _ptr(eps_all), _ptr(x_next), _ptr(cursor_next),
                                            _ptr(n_accept), _ptr(ws), ws.numel(), _stream()), "free_spec_round_finish")
        return x_next, cursor_next, n_accept

    def spec_round_split(self, x_cur, cursor, labels, sched, K, cfg_scale, noise_target, noise_draft, uniforms, rank, world,
                         lam=None, eps_all=None, x_next=None, cursor_next=None, n_accept=None, group=None):
        """One round with the packed pass partitioned over the `world` ranks of a torch.distributed group: begin, an
        all-gather of the noise predictions (every rank contributes the slice it computed; NCCL on GPUs), finish.  Every
        rank must pass identical inputs.  Returns (x_next, cursor_next, n_accept), identical on all ranks."""
        eps_all, lo, hi = self.spec_round_begin(x_cur, cursor, labels, sched, K, cfg_scale, noise_target, noise_draft, uniforms,
                                                rank, world, eps_all=eps_all, lam=lam)
        if world > 1:
            import torch.distributed as dist
            # the rank's own slice is sent from a copy: not every backend takes an input that aliases the output
            dist.all_gather_into_tensor(eps_all, eps_all[lo:hi].clone(), group=group)
        return self.spec_round_finish(eps_all, labels, sched, K, cfg_scale, noise_target, noise_draft, uniforms, x_cur, lam=lam,
                                      x_next=x_next, cursor_next=cursor_next, n_accept=n_accept)

    @staticmethod
    def guided(cfg_scale: float) -> int:
        return 2 if (cfg_scale > 0 and cfg_scale != 1.0) else 1

    def dit_verify_pass(self, x, t_idx, labels, cfg_scale, sched: DeviceSchedule, want_eps=False, want_feat=False,
                        mean_out=None):
        """One packed target pass.  x: CUDA fp32 [n, C, H, W]; t_idx, labels: int32 [n].
        Returns mean [n,C,H,W] (+ eps, + feat [n,G,n_tok,D] when asked)."""
        sh = self.shape
        n = x.shape[0]
        _dev(x, torch.float32); _dev(t_idx, torch.int32); _dev(labels, torch.int32)
        mean = torch.empty_like(x) if mean_out is None else mean_out
        eps = torch.empty_like(x) if want_eps else None
        feat = (torch.empty((n, self.guided(cfg_scale), sh.n_tok, sh.D), dtype=self.act, device=x.device)
                if want_feat else None)
        ws = self.workspace(n)
        _check(lib().dit_verify_pass(self.ctx, n, _ptr(x), _ptr(t_idx), _ptr(labels), float(cfg_scale),
                                     C.byref(sched.desc), _ptr(mean), _ptr(eps), _ptr(feat),
                                     _ptr(ws), ws.numel(), _stream()), "dit_verify_pass")
        out = (mean,) + ((eps,) if want_eps else ()) + ((feat,) if want_feat else ())
        return out if len(out) > 1 else mean

    def dit_verify_pass_raw(self, x, t_idx, labels, guidance: bool, sched: DeviceSchedule, want_feat=False):
        """The packed target pass stopped at the network output: returns eps [n, G, C, H, W] (+ feat)."""
        sh = self.shape
        n, G = x.shape[0], 2 if guidance else 1
        _dev(x, torch.float32); _dev(t_idx, torch.int32); _dev(labels, torch.int32)
        head = torch.empty((n, G, sh.C, sh.H, sh.W), dtype=torch.float32, device=x.device)
        feat = torch.empty((n, G, sh.n_tok, sh.D), dtype=self.act, device=x.device) if want_feat else None
        ws = self.workspace(n)
        _check(lib().dit_verify_pass_raw(self.ctx, n, _ptr(x), _ptr(t_idx), _ptr(labels), int(bool(guidance)),
                                         C.byref(sched.desc), _ptr(head), _ptr(feat), _ptr(ws), ws.numel(), _stream()),
               "dit_verify_pass_raw")
        return (head, feat) if want_feat else head

    def draft_step(self, x_prev, f_prev, t_idx, labels, cfg_scale, sched: DeviceSchedule, noise):
        """One drafter step.  Returns (m_hat, x_hat, f_next)."""
        n = x_prev.shape[0]
        _dev(x_prev, torch.float32); _dev(f_prev, self.act); _dev(noise, torch.float32)
        m_hat, x_hat, f_next = torch.empty_like(x_prev), torch.empty_like(x_prev), torch.empty_like(f_prev)
        ws = self.workspace(n)
        _check(lib().draft_step(self.ctx, n, _ptr(x_prev), _ptr(f_prev), _ptr(_dev(t_idx, torch.int32)),
                                _ptr(_dev(labels, torch.int32)), float(cfg_scale), C.byref(sched.desc), _ptr(noise),
                                _ptr(m_hat), _ptr(x_hat), _ptr(f_next), _ptr(ws), ws.numel(), _stream()), "draft_step")
        return m_hat, x_hat, f_next

    def uncertainty_profile(self, x0, labels, sched: DeviceSchedule, K, cfg_scale, noise_target, noise_draft, uniforms, lam=None):
        """The offline run of Sec. 3.4.  Returns (eps_delta [N], accept_prob [N], count [N]) as numpy arrays."""
        B, N = x0.shape[0], sched.desc.N
        _dev(x0, torch.float32); _dev(labels, torch.int32); _dev(noise_target, torch.float32)
        prm = SpecParams(int(K), float(cfg_scale), None if lam is None else _dev(lam, torch.float32).data_ptr())
        dev, acc, cnt = np.zeros(N), np.zeros(N), np.zeros(N, np.int64)
        ws = self.workspace(B * max(int(K), 1))
        _check(lib().free_uncertainty_profile(self.ctx, B, _ptr(x0), _ptr(labels), C.byref(sched.desc), C.byref(prm),
                                              _ptr(noise_target), _ptr(noise_draft), _ptr(uniforms),
                                              dev.ctypes.data_as(C.c_void_p), acc.ctypes.data_as(C.c_void_p),
                                              cnt.ctypes.data_as(C.c_void_p), _ptr(ws), ws.numel(), _stream()),
               "free_uncertainty_profile")
        return dev, acc, cnt

    def sample_trajectory(self, x0, labels, sched: DeviceSchedule, K, cfg_scale, noise_target, noise_draft=None,
                          uniforms=None, lam=None, use_graph=False):
        """Algorithm 1 for a batch.  Returns (x_final, stats dict)."""
        B = x0.shape[0]
        _dev(x0, torch.float32); _dev(labels, torch.int32); _dev(noise_target, torch.float32)
        prm = SpecParams(int(K), float(cfg_scale), None if lam is None else _dev(lam, torch.float32).data_ptr(), int(bool(use_graph)))
        st = TrajStats()
        x_final = torch.empty_like(x0)
        ws = self.workspace(B * max(int(K), 1))
        _check(lib().sample_trajectory(self.ctx, B, _ptr(x0), _ptr(labels), C.byref(sched.desc), C.byref(prm),
                                       _ptr(noise_target), _ptr(noise_draft), _ptr(uniforms), _ptr(x_final),
                                       C.byref(st), _ptr(ws), ws.numel(), _stream()), "sample_trajectory")
        stats = {k: getattr(st, k) for k in ("rounds", "target_calls", "draft_calls", "accepted", "rejected",
                                             "parallel_efficiency", "graph_rounds")}
        stats["accept_hist"] = list(st.accept_hist)[:int(K) + 1]
        return x_final, stats


# ------------------------------------------------------------------------------------------ single ops
def op_linear(A, W, bias=None, epilogue=EPI_BIAS, out_dtype=None, resid=None, gate=None, rows_per_seq=1):
    """epilogue(A W^T + bias) with the library's linear-layer kernel (fp32: CUDA cores, bf16: tcgen05)."""
    dtype = FREE_FP32 if A.dtype == torch.float32 else FREE_BF16
    M, K = A.shape
    N = W.shape[0]
    od = dtype if out_dtype is None else out_dtype
    out = None if epilogue == EPI_GATE_RESIDUAL else torch.empty((M, N), dtype=_ACT[od], device=A.device)
    ws = torch.zeros(lib().free_op_linear_workspace_bytes(), dtype=torch.uint8, device=A.device)
    _check(lib().free_op_linear(dtype, epilogue, od, M, N, K, _ptr(A), _ptr(W), _ptr(bias), _ptr(out), _ptr(resid),
                                _ptr(gate), 0 if gate is None else gate.stride(0), rows_per_seq,
                                _ptr(ws), ws.numel(), _stream()), "free_op_linear")
    err = int(ws[:4].view(torch.int32).item())
    if err:
        raise FreeError(-8, f"free_op_linear (device error word {err:#x})")
    return resid if epilogue == EPI_GATE_RESIDUAL else out


def op_ln_modulate(x, shift, scale, rows_per_seq, out_dtype=FREE_FP32):
    M, D = x.shape
    y = torch.empty((M, D), dtype=_ACT[out_dtype], device=x.device)
    _check(lib().free_op_ln_modulate(out_dtype, M, D, rows_per_seq, _ptr(x), _ptr(shift), _ptr(scale),
                                     shift.stride(0), _ptr(y), _stream()), "free_op_ln_modulate")
    return y


def op_attention(qkv, heads):
    """qkv [n_seq, n_tok, 3*D] (split as 3, heads, d_head) -> [n_seq, n_tok, D]."""
    dtype = FREE_FP32 if qkv.dtype == torch.float32 else FREE_BF16
    n_seq, n_tok, D3 = qkv.shape
    D = D3 // 3
    out = torch.empty((n_seq, n_tok, D), dtype=qkv.dtype, device=qkv.device)
    need = lib().free_op_attention_workspace_bytes(dtype, n_seq, n_tok, heads, D // heads)
    ws = torch.zeros(need, dtype=torch.uint8, device=qkv.device)
    _check(lib().free_op_attention(dtype, n_seq, n_tok, heads, D // heads, _ptr(qkv), _ptr(out), _ptr(ws), need, _stream()),
           "free_op_attention")
    err = int(ws[:4].view(torch.int32).item())
    if err:
        raise FreeError(-8, f"free_op_attention (device error word {err:#x})")
    return out


STATIC_ATTN_MAX_ELEMS = 1 << 21


def op_attention_static(qkv, heads):
    """bf16 attention through the entry point that allocates nothing inside the library: its scratch is a fixed
    array in the library's device image (for callers that may not allocate).  qkv [n_seq, n_tok, 3*D] bf16.
    The output tensor and the 4-byte error word are the caller's (allocated here by torch, outside the call)."""
    n_seq, n_tok, D3 = qkv.shape
    D = D3 // 3
    _dev(qkv, torch.bfloat16)
    out = torch.empty((n_seq, n_tok, D), dtype=torch.bfloat16, device=qkv.device)
    err = torch.ones(1, dtype=torch.int32, device=qkv.device)
    _check(lib().free_op_attention_static(n_seq, n_tok, heads, D // heads, _ptr(qkv), _ptr(out), _ptr(err), _stream()),
           "free_op_attention_static")
    if int(err.item()):
        raise FreeError(-8, "free_op_attention_static (device error word set)")
    return out
