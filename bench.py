"""Benchmark of the packed parallel-verification path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload round|verifier|verifier_fused|verifier_sweep|drafter_loss|trajectory|ops] [--impl reference]

One JSON line on stdout (rank 0).  A "step" is one pass of the hot path over one batch of synthetic
input resident in HBM; `e2e` repeats it from pinned HOST buffers with the copies inside the timed
region.  The default workload (one FREE round on the DiT-XL/2-shaped 512^2 model) also reports, from the same
process, the verifier on its own (`verifier_roofline`) and whole trajectories in images/s (`trajectory`), and takes its
per-kernel table in a second pass so that the headline is timed without per-launch events.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
Multi-GPU runs shard whole batches across ranks (weak scaling, no data-path collective).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="default")
    ap.add_argument("--batch", type=int, default=0, help="images per step (0 = workload default)")
    ap.add_argument("--graph", action="store_true", help="trajectory workload: replay the rounds as a CUDA graph")
    ap.add_argument("--res", type=int, default=512, choices=[256, 512], help="trajectory workload: image resolution")
    ap.add_argument("--chunk", type=int, default=0, help="verifier_fused: drafts per early-exit chunk (0 = off)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="default workload: skip the verifier and trajectory measurements")
    ap.add_argument("--split", default="replicas", choices=["replicas", "drafts"],
                    help="round workload on N > 1 GPUs: independent replicas (weak scaling, default) or ONE job whose packed "
                         "pass is partitioned over the ranks with an all-gather of the noise predictions per round (strong scaling)")
    ap.add_argument("--no-launch-overlap", action="store_true", help="launch every kernel fully serialised (no programmatic dependent launch)")
    ap.add_argument("--K", type=int, default=0, help="verifier workloads: drafts per sample (0 = 16)")
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for nm, v in zip(names, r[4:8]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": float(max(power))}


# ------------------------------------------------------------------------------------------------
# workloads: each provides device-resident steps, host-buffer steps, algorithmic work and an oracle sample
# ------------------------------------------------------------------------------------------------
class VerifierWorkload:
    """Largest point of the standalone verifier sweep: d = 4x64x64, K = 16 drafts, B = 256 samples, fp32,
    strict acceptance, target means N(0,1), draft = target + small offset, sigma2 from the 250-step schedule.
    Inputs (805 MB) exceed L2, so consecutive steps cannot be served from cache."""
    name = "verifier sweep point K=16 B=256 d=16384 strict"
    metric, unit, dtype = "verifier HBM GB/s", "GB/s", "f32"

    def __init__(self, batch, rank):
        import torch
        import synth
        import paper_2511_20390_b200 as free
        from paper_2511_20390_b200 import binding
        self.torch, self.free, self.binding = torch, free, binding
        self.B, self.K, self.d = (batch or 256), 16, 16384
        sched = free.respaced_schedule(250)
        s2 = np.tile(sched["sigma2"][np.linspace(240, 20, self.K).astype(int)].astype(np.float32), (self.B, 1))
        m, mh, xh, u = synth.verifier_inputs(1000 + rank, self.B, self.K, self.d, 0.0015, s2)
        self.host = dict(m=m, m_hat=mh, x_hat=xh, sigma2=s2, u=u)
        self.dev = {k: torch.from_numpy(v).cuda() for k, v in self.host.items()}
        self.x_out = torch.empty(self.B, self.d, device="cuda")
        self.n_acc = torch.empty(self.B, dtype=torch.int32, device="cuda")
        self.hv = None
        # algorithmic bytes per sample: read m, m_hat, x_hat once, write one state, plus the [B,K] scalars
        self.bytes_per_step = self.B * (3 * self.K * self.d * 4 + self.d * 4 + 12 * self.K)
        self.units_per_step = self.bytes_per_step / 1e9          # GB
        self.launches_per_step = 1
        self.config = {"workload": self.name, "B": self.B, "K": self.K, "d": self.d,
                       "cache": "inputs larger than L2 (805 MB per step)"}

    def step(self):
        d = self.dev
        self.free.spec_verify(d["m"], d["m_hat"], d["x_hat"], d["sigma2"], d["u"], x_out=self.x_out, n_accept=self.n_acc)

    def host_step(self):
        if self.hv is None:
            self.hv = self.binding.HostVerifier(self.B, self.K, self.d)
            self.hv.load(**self.host)
        self.hv.run()
        return self.hv.h2d_bytes, self.hv.d2h_bytes

    # DRAM bytes (read + write) of one launch at B = 64 from the ncu capture summarised in
    # profiles/spec_verify_kernel_K16_B64.txt; traffic is proportional to the batch
    NCU_DRAM_BYTES_B64 = 217.8e6

    def roofline(self, ms_per_step, peaks):
        ach = self.bytes_per_step / 1e9 / (ms_per_step / 1e3)
        traffic = self.NCU_DRAM_BYTES_B64 * self.B / 64.0 if (self.K, self.d) == (16, 16384) else None
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "kernel": "spec_verify_kernel",
                "peak_source": peaks["source"]}

    def oracle_sample(self):
        from oracle import verify as ov
        nb = 4
        h = self.host
        t0 = time.perf_counter()
        ov.spec_verify(h["m"][:nb], h["m_hat"][:nb], h["x_hat"][:nb], h["sigma2"][:nb], h["u"][:nb])
        dt = time.perf_counter() - t0
        by = nb * (3 * self.K * self.d * 4 + self.d * 4 + 12 * self.K)
        return by / 1e9 / dt, f"{nb} of {self.B} samples of the same batch, full K"


class FusedVerifierWorkload:
    """Verification from the noise predictions of the packed pass (guidance + Eq. ddpm_update + Algorithm 2 in one
    kernel) at the same point of the sweep: 4x64x64 latents, two guidance streams, K = 16, B = 256.
    Inputs (1.1 GB) exceed L2.  Draft means sit about 1.8 sigma from the target means (mixed decisions)."""
    name = "fused verifier K=16 B=256 latent 4x64x64 guidance"
    metric, unit, dtype = "verifier HBM GB/s", "GB/s", "f32"
    shape, G, cfg = (4, 64, 64), 2, 4.0

    def __init__(self, batch, rank, chunk=0):
        import torch
        import synth
        import paper_2511_20390_b200 as free
        self.torch, self.free = torch, free
        self.B, self.K, self.d, self.chunk = (batch or 256), 16, int(np.prod(self.shape)), chunk
        B, K, d = self.B, self.K, self.d
        sched = free.respaced_schedule(250)
        s2 = np.tile(sched["sigma2"][np.linspace(240, 20, K).astype(int)].astype(np.float32), (B, 1))
        sig, ce = float(np.sqrt(s2.mean())), 0.05
        s = 0.35 * sig / np.sqrt(d)
        eps, x_first, mh, xh, u = synth.eps_verifier_inputs(2000 + rank, B, K, self.G, self.shape, s, s2, eps_std=s / ce)
        cx = np.ones((B, K), np.float32)
        self.host = dict(eps=eps, x_first=x_first, m_hat=mh, x_hat=xh, cx=cx, ce=np.full((B, K), ce, np.float32), sigma2=s2, u=u)
        self.dev = {k: torch.from_numpy(v).cuda() for k, v in self.host.items()}
        self.x_out = torch.empty((B,) + self.shape, device="cuda")
        self.n_acc = torch.empty(B, dtype=torch.int32, device="cuda")
        self.pinned = None
        # algorithmic bytes per sample: per draft the noise predictions of both streams, m_hat and x_hat once; the first
        # state and the output once; the [B,K] scalars
        self.bytes_per_step = B * (K * (self.G + 2) * d * 4 + 2 * d * 4 + 20 * K)
        self.units_per_step = self.bytes_per_step / 1e9
        self.launches_per_step = 1
        self.config = {"workload": self.name, "B": B, "K": K, "d": d, "chunk": chunk,
                       "cache": "inputs larger than L2 (1.1 GB per step)"}

    def _call(self, d):
        self.free.spec_verify_fused(d["eps"], d["x_first"], d["m_hat"], d["x_hat"], d["cx"], d["ce"], d["sigma2"], d["u"],
                                    self.cfg, chunk=self.chunk, x_out=self.x_out, n_accept=self.n_acc)

    def step(self):
        self._call(self.dev)

    def host_step(self):
        torch = self.torch
        if self.pinned is None:
            self.pinned = {k: torch.from_numpy(v).pin_memory() for k, v in self.host.items()}
            self.stage = {k: torch.empty_like(v, device="cuda") for k, v in self.pinned.items()}
            self.h_x, self.h_n = torch.empty(self.x_out.shape, pin_memory=True), torch.empty(self.B, dtype=torch.int32, pin_memory=True)
        for k, v in self.pinned.items():
            self.stage[k].copy_(v, non_blocking=True)
        self._call(self.stage)
        self.h_x.copy_(self.x_out, non_blocking=True)
        self.h_n.copy_(self.n_acc, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return (sum(v.numel() * v.element_size() for v in self.pinned.values()),
                self.h_x.numel() * 4 + self.h_n.numel() * 4)

    def bytes_examined(self):
        """With the early exit only whole chunks up to the first rejection are read: the bytes of those rows."""
        if self.chunk <= 0:
            return self.bytes_per_step
        n = self.n_acc.cpu().numpy().astype(np.int64)
        rows = np.minimum(self.K, (np.minimum(n, self.K - 1) // self.chunk + 1) * self.chunk)
        return int((rows * (self.G + 2) * self.d * 4 + 2 * self.d * 4 + 20 * rows).sum())

    # DRAM bytes (read + write) of one launch at B = 64, chunk 0, from the ncu capture summarised in
    # profiles/spec_verify_fused_kernel_K16_B64.txt; traffic is proportional to the batch
    NCU_DRAM_BYTES_B64 = 298.2e6

    def roofline(self, ms_per_step, peaks):
        ach = self.bytes_examined() / 1e9 / (ms_per_step / 1e3)
        traffic = self.NCU_DRAM_BYTES_B64 * self.B / 64.0 if self.chunk == 0 else None
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "kernel": "spec_verify_fused_kernel",
                "peak_source": peaks["source"]}

    def extra(self, ms_step, peaks):
        return {"accepted_per_sample": float(self.n_acc.float().mean().item()),
                "bytes_read_fraction": self.bytes_examined() / self.bytes_per_step}

    def oracle_sample(self):
        from oracle import verify as ov
        nb, h = 2, self.host
        t0 = time.perf_counter()
        ov.spec_verify_from_eps(h["eps"][:nb], h["x_first"][:nb], h["m_hat"][:nb], h["x_hat"][:nb], h["cx"][:nb], h["ce"][:nb],
                                self.cfg, h["sigma2"][:nb], h["u"][:nb])
        dt = time.perf_counter() - t0
        return nb * self.bytes_per_step / self.B / 1e9 / dt, f"{nb} of {self.B} samples of the same batch, full K"


class DrafterLossWorkload:
    """The drafter's training objectives (Sec. 3.2) on DiT-XL/2 512^2 shapes: per sample a bf16 top-block feature pair
    [1024, 1152] and an fp32 noise pair [4, 64, 64]; 256 samples per step (1.24 GB, larger than L2)."""
    name = "drafter loss, 256 samples, features [1024, 1152] bf16, noise 4x64x64"
    metric, unit, dtype = "loss reduction HBM GB/s", "GB/s", "f32"

    def __init__(self, batch, rank):
        import torch
        import paper_2511_20390_b200 as free
        self.torch, self.free = torch, free
        self.n, self.n_tok, self.D, self.d_eps = (batch or 256), 1024, 1152, 16384
        g = torch.Generator(device="cuda"); g.manual_seed(3000 + rank)
        mk = lambda *s: torch.randn(*s, generator=g, device="cuda", dtype=torch.float32)
        self.f_ref = mk(self.n, self.n_tok, self.D).bfloat16()
        self.f_pred = (self.f_ref.float() + 0.3 * mk(self.n, self.n_tok, self.D)).bfloat16()
        self.e_ref = mk(self.n, self.d_eps)
        self.e_pred = self.e_ref + 0.1 * mk(self.n, self.d_eps)
        self.out = torch.empty(4, dtype=torch.float64, device="cuda")
        self.bytes_per_step = 2 * self.n * self.n_tok * self.D * 2 + 2 * self.n * self.d_eps * 4
        self.units_per_step = self.bytes_per_step / 1e9
        self.launches_per_step = 2
        self.pinned = None
        self.config = {"workload": self.name, "samples": self.n, "cache": "inputs larger than L2 (1.24 GB per step)"}

    def step(self):
        self.free.drafter_loss(self.e_pred, self.e_ref, self.f_pred, self.f_ref, 0.5, 0.01, out=self.out)

    def host_step(self):
        torch = self.torch
        if self.pinned is None:
            self.pinned = [t.cpu().pin_memory() for t in (self.e_pred, self.e_ref, self.f_pred, self.f_ref)]
            self.stage = [torch.empty_like(t, device="cuda") for t in self.pinned]
            self.h_out = torch.empty(4, dtype=torch.float64, pin_memory=True)
        for d, h in zip(self.stage, self.pinned):
            d.copy_(h, non_blocking=True)
        self.free.drafter_loss(*self.stage, 0.5, 0.01, out=self.out)
        self.h_out.copy_(self.out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return sum(t.numel() * t.element_size() for t in self.pinned), 32

    # DRAM bytes (read + write) of one launch at 64 samples from the ncu capture summarised in
    # profiles/loss_partial_kernel_xl512_64samples.txt; traffic is proportional to the batch
    NCU_DRAM_BYTES_64 = 313.7e6

    def roofline(self, ms_per_step, peaks):
        ach = self.bytes_per_step / 1e9 / (ms_per_step / 1e3)
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "traffic": self.NCU_DRAM_BYTES_64 * self.n / 64.0, "kernel": "loss_partial_kernel", "peak_source": peaks["source"]}

    def oracle_sample(self):
        from oracle import losses as ol
        nb = 8
        a = [t[:nb].float().cpu().numpy() for t in (self.e_pred, self.e_ref, self.f_pred, self.f_ref)]
        t0 = time.perf_counter()
        ol.free_loss(*a, 0.5, 0.01)
        dt = time.perf_counter() - t0
        return nb * self.bytes_per_step / self.n / 1e9 / dt, f"{nb} of {self.n} samples of the same batch"


def make_workload(name, batch, rank, chunk=0, split=None):
    if name == "drafter_loss":
        return DrafterLossWorkload(batch, rank)
    if name in ("verifier",):
        return VerifierWorkload(batch, rank)
    if name == "verifier_fused":
        return FusedVerifierWorkload(batch, rank, chunk)
    if name in ("default", "round"):
        try:
            from bench_round import RoundWorkload        # the full packed-verify round (DiT + verifier)
        except ImportError:
            return VerifierWorkload(batch, rank)
        return RoundWorkload(batch, rank, split=split)
    if name == "ops":
        from bench_round import OpsWorkload
        return OpsWorkload(batch, rank)
    raise SystemExit(f"unknown workload {name}")


def time_launches(fn, launches=20, warm=3):
    """Mean device time (ms) of `launches` calls of fn on the current stream, CUDA events, after `warm` calls."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(launches):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / launches


def time_launches_graph(fn, launches=20, warm=3):
    """As time_launches, with the `launches` calls recorded into one CUDA graph and the replay timed: the device time of
    short kernels, free of the host's launch rate."""
    import torch
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for _ in range(launches):
                fn()
        graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / launches


def verifier_extras(peaks, launches=20):
    """The verifier on its own at the largest point of the sweep (K = 16, B = 256, latent 4x64x64; inputs of 0.8 / 1.1 GB,
    larger than L2): from means (spec_verify) and from the noise predictions (spec_verify_fused)."""
    import gc
    import torch
    out = {}
    for key, cls in (("standalone", VerifierWorkload), ("fused", FusedVerifierWorkload)):
        wl = cls(0, 0)
        ms = time_launches(wl.step, launches)
        r = wl.roofline(ms, peaks)
        out[key] = {"kernel": r["kernel"], "bound": "hbm", "achieved": r["achieved"], "peak": r["peak"], "unit": "GB/s", "frac": r["frac"],
                    "traffic": r["traffic"], "ms_per_launch": ms, "launches": launches, "bytes_per_launch": wl.bytes_per_step,
                    "workload": wl.name}
        del wl
        gc.collect(); torch.cuda.empty_cache()
    out["peak_source"] = peaks["source"] + " (copy bandwidth)"
    return out


def verifier_sweep(args, peaks):
    """`--workload verifier_sweep`: GB/s and fraction of the measured copy bandwidth of spec_verify over the sweep of
    drafts per sample, batch and acceptance mode (latent 4x64x64).  Points whose inputs fit L2 are marked: their figure is
    a cache figure, not an HBM one."""
    import torch
    import synth
    import paper_2511_20390_b200 as free
    d = 16384
    sched = free.respaced_schedule(250)
    rows = []
    for K in ([args.K] if args.K else [2, 4, 6, 8, 16]):
        for B in ([args.batch] if args.batch else [1, 4, 16, 64, 256]):
            s2 = np.tile(sched["sigma2"][np.linspace(240, 20, K).astype(int)].astype(np.float32), (B, 1))
            m, mh, xh, u = synth.verifier_inputs(4000 + K, B, K, d, 0.0015, s2)
            dev = [torch.from_numpy(a).cuda() for a in (m, mh, xh, s2, u)]
            lam = torch.full((B, K), 0.5, device="cuda")
            x_out, n_acc = torch.empty(B, d, device="cuda"), torch.empty(B, dtype=torch.int32, device="cuda")
            by = B * (3 * K * d * 4 + d * 4 + 12 * K)
            for mode, lm in (("strict", None), ("relaxed", lam)):
                ms = time_launches_graph(lambda: free.spec_verify(*dev, lam=lm, x_out=x_out, n_accept=n_acc), 20)
                gbs = by / 1e9 / (ms / 1e3)
                rows.append({"K": K, "B": B, "mode": mode, "us": round(ms * 1e3, 2), "gbs": round(gbs, 1),
                             "frac_of_copy": round(gbs / peaks["hbm_gbs"], 4), "MB": round(by / 1e6, 2),
                             "fits_l2": by < 126e6})
    print(json.dumps({"metric": "verifier HBM GB/s", "unit": "GB/s", "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
                      "config": {"workload": "spec_verify sweep, latent 4x64x64, 20 launches per point replayed as one CUDA graph after 3 warm-ups"},
                      "points": rows}))


def max_over_ranks(times_ms, device):
    """Element-wise maximum of per-rank timings over all ranks (every rank gets the result); single process: identity.
    The job's time is that of its slowest rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(t) for t in times_ms]
    t = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(units_per_rank_step, world, ms_per_step):
    """Aggregate throughput of `world` ranks that each process `units_per_rank_step` per step (weak scaling)."""
    return units_per_rank_step * world / (ms_per_step / 1e3)


def cpu_threads():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, rank):
    """The CPU oracle, as it stands, on a bounded sample of the workload per step."""
    if rank != 0:
        return
    os.environ.setdefault("CUDA_VISIBLE_DEVICES", "")
    wl_name = args.workload
    # the oracle needs no GPU: build host inputs only
    import synth
    from oracle import verify as ov
    import importlib
    cores = cpu_threads()
    try:
        br = importlib.import_module("bench_round")
        out = br.reference_arm(args, cores)
    except ImportError:
        from paper_2511_20390_b200.schedule import respaced_schedule
        B, K, d, nb = 256, 16, 16384, 2
        s2 = np.tile(respaced_schedule(250)["sigma2"][np.linspace(240, 20, K).astype(int)].astype(np.float32), (nb, 1))
        m, mh, xh, u = synth.verifier_inputs(1000, nb, K, d, 0.0015, s2)
        by = nb * (3 * K * d * 4 + d * 4 + 12 * K)
        for _ in range(args.warmup):
            ov.spec_verify(m, mh, xh, s2, u)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            ov.spec_verify(m, mh, xh, s2, u)
        dt = (time.perf_counter() - t0) / args.steps
        val = by / 1e9 / dt
        out = {"metric": VerifierWorkload.metric, "value": val, "unit": "GB/s", "ms_per_step": dt * 1e3,
               "dtype": "f64", "config": {"workload": VerifierWorkload.name},
               "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "sample": f"{nb} of {B} samples per step"}}
    out.update({"impl": "reference", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "data": "synthetic",
                "gpu_launches": 0})
    out["e2e"] = {"value": out["value"], "unit": out["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    print(json.dumps(out))


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        return run_reference(args, rank)

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    import paper_2511_20390_b200 as free
    free.lib()        # fail loudly if the CUDA library is not built
    if args.no_launch_overlap:
        free.lib().free_set_launch_overlap(0)
    if args.workload == "trajectory":     # whole trajectories have their own protocol (one step takes tens of seconds)
        if rank == 0:
            from bench_round import run_trajectory
            run_trajectory(args)
        return

    peaks = measured_peaks()
    if args.workload == "verifier_sweep":
        if rank == 0:
            verifier_sweep(args, peaks)
        return
    split = (rank, world) if args.split == "drafts" and args.workload in ("default", "round") else None
    wl = make_workload(args.workload, args.batch, rank, args.chunk, split)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        wl.step()
    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        wl.step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    if hasattr(wl, "begin_timed"):
        # second pass of the same steps with CUDA events around every kernel launch (the per-kernel table and the
        # roofline of the dominant kernel); the headline above is timed without them
        wl.begin_timed()
        for _ in range(args.steps):
            wl.step()
        wl.end_timed(args.steps)
        barrier()
    kernel_ms = wl.kernel_ms_per_launch() if hasattr(wl, "kernel_ms_per_launch") else ms / args.steps
    clocks = sampler.stop() if sampler else None

    # end to end from pinned host buffers
    for _ in range(2):
        wl.host_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_e2e = max(2, min(args.steps, 20))          # as many steps as the device-resident timing, so that the two compare
    e0.record(stream)
    for _ in range(n_e2e):
        h2d, d2h = wl.host_step()
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1)

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], "cuda")
    ms_step = ms / args.steps
    # replicas: every rank processed its own batch; a partitioned job: the ranks shared one batch
    ranks_of_work = 1 if getattr(wl, "scaling", "weak") == "strong" else world
    value = whole_job_value(wl.units_per_step, ranks_of_work, ms_step)
    e2e_value = whole_job_value(wl.units_per_step, ranks_of_work, ms_e2e / n_e2e)

    if rank == 0:
        out = {"metric": wl.metric, "value": value, "unit": wl.unit, "n_gpus": world, "steps": args.steps,
               "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": getattr(wl, "scaling", "weak"),
               "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic", "config": wl.config,
               "clocks": clocks,
               "e2e": {"value": e2e_value, "unit": wl.unit, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
               "gpu_launches": int(round(wl.launches_per_step * args.steps)),
               "roofline": wl.roofline(kernel_ms, peaks)}
        if hasattr(wl, "extra"):
            out.update(wl.extra(ms_step, dict(peaks, sm_mhz=clocks["sm_mhz"] if clocks else None)))
        if world == 1 and args.workload == "default" and not args.no_extras:
            # the other two parts of the metric, measured in this process: verifier HBM GB/s and images/s
            if hasattr(wl, "trajectory_extras"):
                out["trajectory"] = wl.trajectory_extras()
                out["latency_b1"] = wl.latency_extras()
            out["verifier_roofline"] = verifier_extras(peaks)
        if world == 1 and not args.no_cpu_baseline:
            v, sample = wl.oracle_sample()
            out["cpu_baseline"] = {"value": v, "unit": wl.unit, "cores": cpu_threads(), "kind": "oracle", "sample": sample}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
