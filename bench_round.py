"""The benchmark's main workload: one speculative round of FREE on a DiT-XL/2-shaped model at 512^2.

Step = the whole hot path once for a batch of B images (Algorithm 1's loop body): target step on the B current
latents, K = 6 drafter steps, ONE packed target pass over B*K states (each doubled by classifier-free guidance),
the fused verifier, the cursor update.  Weights are random-init (no checkpoints exist here), latents N(0,1),
labels uniform over 1000 classes, 250-step respaced DDPM schedule.
"""
import os
import time

import numpy as np

K_DRAFTS, CFG, N_SCHED = 6, 4.0, 250


def round_flops(shape, B, K, G, n_draft_blocks=1):
    """Algorithmic FLOPs of one round: 2MNK per linear layer + 4 T^2 d_head per (head, block, sequence);
    target step (B*G sequences), K drafter steps (fusion layer + blocks), packed pass (B*K*G sequences)."""
    seq = shape.flops_per_sequence()
    fuse = 2.0 * shape.n_tok * shape.D * 2 * shape.D
    draft = shape.flops_per_sequence(depth=n_draft_blocks) + fuse
    return B * G * seq + K * B * G * draft + B * K * G * seq


def round_config(B, K, G):
    """The `config` object of the round workload (shared by the CUDA arm and the oracle arm of the benchmark)."""
    return {"workload": f"FREE round, DiT-XL/2-shaped 512^2 (latent 4x64x64, 1024 tokens, width 1152, 28 blocks, "
                        f"16 heads), K={K} drafts, cfg {CFG} (doubled batch), batch {B}, 1-block drafter, "
                        f"{N_SCHED}-step schedule",
            "B": B, "K": K, "sequences_in_packed_pass": B * K * G,
            "cache": "activations per step (several GB) exceed L2"}


class RoundWorkload:
    metric = "DiT-XL/2 512^2 packed-verify TFLOP/s"
    unit = "TFLOP/s"
    dtype = "bf16"

    scaling = "weak"

    def __init__(self, batch, rank, split=None):
        """split = (rank, world): ONE job whose packed pass is partitioned over the ranks (the paper's deployment, Sec. 4:
        drafts verified on parallel GPUs); every rank then holds the same weights and inputs, and the job's work does not
        grow with the number of ranks (strong scaling).  Default: every rank runs its own batch (replicas)."""
        import torch
        import synth
        import paper_2511_20390_b200 as free
        self.torch, self.free = torch, free
        self.shape = synth.DIT_XL2_512
        self.B = batch or 16
        self.split = split
        if split:
            rank, self.scaling = 0, "strong"          # identical seeds on every rank
        B, K, sh = self.B, K_DRAFTS, self.shape
        self.model = free.Model.random(sh, 1234 + rank, dtype="bf16", with_drafter=True)
        self.sched = free.DeviceSchedule(free.respaced_schedule(N_SCHED))
        g = torch.Generator(device="cuda")
        g.manual_seed(99 + rank)
        d = sh.d_latent
        rn = lambda *s: torch.randn(*s, generator=g, device="cuda", dtype=torch.float32)
        self.x_cur = rn(B, sh.C, sh.H, sh.W)
        self.labels = torch.randint(0, sh.n_classes, (B,), generator=g, device="cuda", dtype=torch.int32)
        # every step restarts from the same cursor (transition 21 of 250), so all steps do identical work
        self.cursor = torch.full((B,), 21, dtype=torch.int32, device="cuda")
        self.noise_t, self.noise_d = rn(B, N_SCHED, d), rn(B, N_SCHED, d)
        self.uniforms = torch.rand(B, N_SCHED, generator=g, device="cuda", dtype=torch.float32)
        self.x_next = torch.empty_like(self.x_cur)
        self.cursor_next = torch.empty_like(self.cursor)
        self.n_acc = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.G = 2
        self.flops = round_flops(sh, B, K, self.G)
        self.units_per_step = self.flops / 1e12
        self.config = round_config(B, K, self.G)
        if split:
            self.config["parallelism"] = (f"packed pass partitioned over {split[1]} ranks ({B * K // split[1]} of {B * K} states each), "
                                          "target step, drafter and verifier replicated, one all-gather of the noise predictions per round")
            self.eps_all = torch.empty((B * K, self.G, sh.C, sh.H, sh.W), dtype=torch.float32, device="cuda")
        # host staging for the end-to-end path: everything one round consumes.  From cursor a = 21 the round takes the
        # target's noise of transition 21 (row 20), the drafter's noise of transitions 22..27 (rows 21..26) and the
        # uniforms of the same six transitions
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        a0 = 20
        self.rows_t, self.rows_d = slice(a0, a0 + 1), slice(a0 + 1, a0 + 1 + K)
        self.h_in = [pin(self.x_cur), pin(self.cursor), pin(self.labels)]
        self.h_zt = [pin(self.noise_t[b, self.rows_t]) for b in range(B)]
        self.h_zd = [pin(self.noise_d[b, self.rows_d]) for b in range(B)]
        self.h_u = pin(self.uniforms)                  # [B, N] is 16 KB: the whole table travels
        self.h_out = [torch.empty(self.x_next.shape, dtype=torch.float32, pin_memory=True),
                      torch.empty(B, dtype=torch.int32, pin_memory=True), torch.empty(B, dtype=torch.int32, pin_memory=True)]
        self.launches_per_step = None
        self._prof = None

    def _round(self):
        if self.split:
            self.model.spec_round_split(self.x_cur, self.cursor, self.labels, self.sched, K_DRAFTS, CFG, self.noise_t, self.noise_d,
                                        self.uniforms, self.split[0], self.split[1], eps_all=self.eps_all, x_next=self.x_next,
                                        cursor_next=self.cursor_next, n_accept=self.n_acc)
            return
        self.model.spec_round(self.x_cur, self.cursor, self.labels, self.sched, K_DRAFTS, CFG, self.noise_t, self.noise_d,
                              self.uniforms, x_next=self.x_next, cursor_next=self.cursor_next, n_accept=self.n_acc)

    def begin_timed(self):
        self.model.profile_begin()

    def end_timed(self, steps):
        self._prof = self.model.profile_end()
        self.launches_per_step = sum(p["launches"] for p in self._prof) / steps
        err = self.model.device_error()
        if err:
            raise RuntimeError(f"device error word {err:#x}: a bounded wait gave up, the timing is void")

    def step(self):
        self._round()

    def host_step(self):
        self.x_cur.copy_(self.h_in[0], non_blocking=True)
        self.cursor.copy_(self.h_in[1], non_blocking=True)
        self.labels.copy_(self.h_in[2], non_blocking=True)
        for b in range(self.B):                        # contiguous row runs: one plain asynchronous copy each
            self.noise_t[b, self.rows_t].copy_(self.h_zt[b], non_blocking=True)
            self.noise_d[b, self.rows_d].copy_(self.h_zd[b], non_blocking=True)
        self.uniforms.copy_(self.h_u, non_blocking=True)
        self._round()
        self.h_out[0].copy_(self.x_next, non_blocking=True)
        self.h_out[1].copy_(self.cursor_next, non_blocking=True)
        self.h_out[2].copy_(self.n_acc, non_blocking=True)
        h2d = sum(x.numel() * x.element_size() for x in self.h_in + self.h_zt + self.h_zd + [self.h_u])
        d2h = sum(x.numel() * x.element_size() for x in self.h_out)
        return h2d, d2h

    def kernel_ms_per_launch(self):
        return None

    # DRAM bytes (read + write) of one fc1 launch at 24 sequences from the ncu capture summarised in
    # profiles/linear_tc2_kernel_xl_block_24seq.txt; None when the kernel changed after the capture
    NCU_FC1_DRAM_BYTES_24SEQ = 240.66e6

    def roofline(self, _ms, peaks):
        """Dominant kernel = the CTA-pair linear kernel (qkv, proj, fc1, fc2 launches of every pass): algorithmic
        2 M N K of its launches over their summed device time (CUDA events inside the timed region)."""
        lin = [p for p in self._prof if p["name"].startswith("linear")]
        ms = sum(p["ms"] for p in lin)
        work = sum(p["work"] for p in lin)
        launches = sum(p["launches"] for p in lin)
        ach = work / 1e12 / (ms / 1e3)
        peak = peaks["bf16_tflops_sustained"]
        top = max(lin, key=lambda p: p["ms"])
        traffic = None
        if self.NCU_FC1_DRAM_BYTES_24SEQ is not None:
            # traffic of the 192-sequence fc1 launch of the packed pass: proportional to M at fixed N, K
            traffic = self.NCU_FC1_DRAM_BYTES_24SEQ * (self.B * K_DRAFTS * self.G / 24.0)
        return {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                "traffic": traffic, "traffic_of": "fc1 launch of the packed pass (scaled from a 24-sequence ncu capture)",
                "kernel": "linear_tc2_kernel (qkv, proj, fc1, fc2)", "launches": launches,
                "ms_per_launch": ms / launches, "largest_class": top["name"],
                "peak_source": peaks["source"] + " (sustained bf16 GEMM)"}

    def extra(self, ms_step, peaks):
        tot = sum(p["ms"] for p in self._prof)
        kern = []
        for p in sorted(self._prof, key=lambda p: -p["ms"]):
            e = {"name": p["name"], "launches": p["launches"], "ms": round(p["ms"], 3), "share": round(p["ms"] / tot, 4)}
            if p["name"].startswith(("linear", "attention", "drafter", "head", "conditioning")) and p["ms"] > 0:
                e["tflops"] = round(p["work"] / 1e12 / (p["ms"] / 1e3), 1)
            elif p["work"] > 0 and p["ms"] > 0:
                e["gbs"] = round(p["work"] / 1e9 / (p["ms"] / 1e3), 1)
            kern.append(e)
        value = self.flops / 1e12 / (ms_step / 1e3)
        more = {}
        att = next((e for e in kern if e["name"] == "attention" and "tflops" in e), None)
        if att and peaks.get("sm_mhz"):
            # attention at d_head 72 is bounded by the exp2 unit, not the tensor core: 16 exponentials per clock per SM,
            # one per score, and a score stands for 4 d_head algorithmic FLOPs (its share of Q K^T and of P V)
            n_sm = self.torch.cuda.get_device_properties(0).multi_processor_count
            peak = 16.0 * n_sm * peaks["sm_mhz"] * 1e6 * 4.0 * self.shape.d_head / 1e12
            more["attention_roofline"] = {"bound": "alu", "achieved": att["tflops"], "peak": round(peak, 1), "unit": "TFLOP/s",
                                          "frac": round(att["tflops"] / peak, 4), "kernel": "attention_tc2_kernel",
                                          "peak_source": "exp2 unit: 16 per clock per SM x SMs x median SM clock of this run x 4 d_head FLOP"}
        return {**more, "pct_of_bf16_peak": {"of_measured_sustained": value / peaks["bf16_tflops_sustained"],
                                     "of_measured_burst": value / peaks["bf16_tflops"], "of_nominal_2250": value / 2250.0},
                "images_per_s_if_all_accepted": self.B * (K_DRAFTS + 1) / N_SCHED / (ms_step / 1e3),
                "kernels": kern}

    def trajectory_extras(self):
        """images/s of whole 250-transition trajectories with this workload's model and batch: every draft accepted
        (u = 0: the most a round can finalise) and the sequential sampler (K = 0) on the same GPU."""
        out = time_trajectories(self.model, self.shape, self.B, {"all_accepted": (K_DRAFTS, 0.0), "sequential_K0": (0, None)}, warm=False)
        return {"unit": "images/s", "api": "sample_trajectory", "transitions": N_SCHED, "batch": self.B, "K": K_DRAFTS,
                "timing": "CUDA events around the blocking call (one host synchronisation per round inside)", **out}

    def latency_extras(self):
        """Batch 1 (the regime where a single step under-fills the GPU): milliseconds per sequential step (K = 0) and per
        speculative round (K = 6, every draft accepted) of whole 250-transition trajectories, launched kernel by kernel
        and with the rounds replayed as a CUDA graph."""
        out = {"unit": "ms", "batch": 1, "api": "sample_trajectory"}
        for mode, graph in (("eager", False), ("graph", True)):
            r = time_trajectories(self.model, self.shape, 1, {"all_accepted": (K_DRAFTS, 0.0), "sequential_K0": (0, None)},
                                  use_graph=graph, warm=False)
            out[mode] = {"ms_per_sequential_step": 1e3 * r["sequential_K0"]["seconds"] / r["sequential_K0"]["rounds"],
                         "ms_per_round": 1e3 * r["all_accepted"]["seconds"] / r["all_accepted"]["rounds"],
                         "seconds_per_image_sequential": r["sequential_K0"]["seconds"],
                         "seconds_per_image_all_accepted": r["all_accepted"]["seconds"],
                         "graph_rounds": r["all_accepted"]["graph_rounds"] + r["sequential_K0"]["graph_rounds"]}
        return out

    def oracle_sample(self):
        return oracle_dit_sample(self.shape)


def oracle_dit_sample(shape, n_blocks=3):
    """Times the fp64 oracle on one sequence through `n_blocks` of the 28 blocks (plus embedding and head)."""
    import dataclasses
    import synth
    from oracle import dit as odit
    sh = dataclasses.replace(shape, depth=n_blocks)
    w = synth.make_target_weights(sh, 5, bf16=True)
    x = synth.normal(5, 77, (sh.C, sh.H, sh.W))
    t0 = time.perf_counter()
    odit.forward(w, sh, x, 500.0, 7)
    dt = time.perf_counter() - t0
    return sh.flops_per_sequence() / 1e12 / dt, f"1 sequence (1024 tokens) through {n_blocks} of 28 blocks, fp64 numpy"


def reference_arm(args, cores):
    """bench.py --impl reference: the oracle as it stands, one bounded sample per step."""
    import synth
    shape = synth.DIT_XL2_512
    vals = []
    for _ in range(min(args.warmup, 1)):
        oracle_dit_sample(shape, 1)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        v, sample = oracle_dit_sample(shape, 2)
        vals.append(v)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    val = float(np.mean(vals))
    return {"metric": RoundWorkload.metric, "value": val, "unit": "TFLOP/s", "ms_per_step": dt * 1e3, "dtype": "f64",
            "config": round_config(args.batch or 16, K_DRAFTS, 2),
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}}


class OpsWorkload:
    """The hot kernels of one DiT-XL/2 block on their own, at 24 sequences of 1024 tokens (M = 24576 rows):
    LayerNorm+modulate, QKV GEMM (head-major scatter is exercised by the full pass; here plain bias), attention,
    proj GEMM (+gate, residual), fc1 GEMM (+GELU), fc2 GEMM (+gate, residual).  Used for profiling single kernels
    on a case small enough for a full counter capture (inputs still exceed L2)."""
    metric, unit, dtype = "DiT-XL/2 block kernels TFLOP/s", "TFLOP/s", "bf16"

    def __init__(self, batch, rank):
        import torch
        from paper_2511_20390_b200 import binding as b
        self.torch, self.b = torch, b
        S, T, D, h = (batch or 24), 1024, 1152, 16
        self.S, self.T, self.D, self.h = S, T, D, h
        M, F = S * T, 4 * D
        g = torch.Generator(device="cuda"); g.manual_seed(5 + rank)
        rn = lambda *s, std=1.0: torch.randn(*s, generator=g, device="cuda") * std
        self.x = rn(M, D)
        self.mod = rn(S, 6 * D, std=0.1)
        self.hn = rn(M, D).bfloat16()
        self.qkv = rn(S, T, 3 * D).bfloat16()
        self.hm = rn(M, F).bfloat16()
        self.w = {k: rn(*s, std=0.02).bfloat16() for k, s in (("qkv", (3 * D, D)), ("proj", (D, D)), ("fc1", (F, D)), ("fc2", (D, F)))}
        self.bias = {k: rn(v.shape[0], std=0.02) for k, v in self.w.items()}
        self.flops = 2.0 * M * D * (3 * D + D + 2 * F) + 4.0 * S * h * T * T * (D // h)
        self.units_per_step = self.flops / 1e12
        self.launches_per_step = 6
        self.config = {"workload": f"one DiT-XL/2 block's kernels, {S} sequences x 1024 tokens", "cache": "operands exceed L2"}

    def step(self):
        b = self.b
        D = self.D
        b.op_ln_modulate(self.x, self.mod[:, :D], self.mod[:, D:2 * D], self.T, out_dtype=b.FREE_BF16)
        b.op_linear(self.hn, self.w["qkv"], self.bias["qkv"])
        att = b.op_attention(self.qkv, self.h)
        b.op_linear(att.view(-1, D), self.w["proj"], self.bias["proj"], epilogue=b.EPI_GATE_RESIDUAL, resid=self.x,
                    gate=self.mod[:, 2 * D:3 * D], rows_per_seq=self.T)
        b.op_linear(self.hn, self.w["fc1"], self.bias["fc1"], epilogue=b.EPI_BIAS_GELU)
        b.op_linear(self.hm, self.w["fc2"], self.bias["fc2"], epilogue=b.EPI_GATE_RESIDUAL, resid=self.x,
                    gate=self.mod[:, 5 * D:6 * D], rows_per_seq=self.T)

    def host_step(self):
        self.step()
        return 0, 0

    def roofline(self, ms, peaks):
        ach = self.flops / 1e12 / (ms / 1e3)
        return {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
                "traffic": None, "kernel": "block kernels (aggregate)", "peak_source": peaks["source"]}

    def oracle_sample(self):
        import synth
        return oracle_dit_sample(synth.DIT_XL2_512, 1)


def time_trajectories(model, sh, B, regimes, seed=7, use_graph=False, warm=True):
    """Whole sampling trajectories through sample_trajectory (Algorithm 1 end to end; the call blocks and synchronises
    once per round): device time by CUDA events around each call.  `regimes`: name -> (K, uniforms or a constant or None)."""
    import torch
    import paper_2511_20390_b200 as free
    sched = free.DeviceSchedule(free.respaced_schedule(N_SCHED))
    g = torch.Generator(device="cuda"); g.manual_seed(seed)
    d = sh.d_latent
    rn = lambda *s_: torch.randn(*s_, generator=g, device="cuda", dtype=torch.float32)
    x0 = rn(B, sh.C, sh.H, sh.W)
    labels = torch.randint(0, sh.n_classes, (B,), generator=g, device="cuda", dtype=torch.int32)
    zt, zd = rn(B, N_SCHED, d), rn(B, N_SCHED, d)
    uni = {}
    for name, (K, u) in regimes.items():
        if u == "seeded":
            u = torch.rand(B, N_SCHED, generator=g, device="cuda")
        elif u is not None:
            u = torch.full((B, N_SCHED), float(u), device="cuda")
        uni[name] = u
    if warm:
        model.sample_trajectory(x0, labels, sched, K_DRAFTS, CFG, zt, zd, torch.zeros(B, N_SCHED, device="cuda"))
        torch.cuda.synchronize()
    out = {}
    side = torch.cuda.Stream()            # the legacy default stream cannot be captured into a graph
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for name, (K, _) in regimes.items():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            x, st = model.sample_trajectory(x0, labels, sched, K, CFG, zt, zd if K else None, uni[name], use_graph=use_graph)
            e1.record()
            torch.cuda.synchronize()
            sec = e0.elapsed_time(e1) / 1e3
            assert torch.isfinite(x).all()
            out[name] = {"images_per_s": B / sec, "seconds": sec, "rounds": st["rounds"], "target_calls": st["target_calls"],
                         "draft_calls": st["draft_calls"], "accepted": st["accepted"], "rejected": st["rejected"],
                         "parallel_efficiency": st["parallel_efficiency"], "graph_rounds": st["graph_rounds"]}
    torch.cuda.current_stream().wait_stream(side)
    return out


def run_trajectory(args):
    """`bench.py --workload trajectory`: whole sampling trajectories (Algorithm 1 end to end through sample_trajectory)
    on the DiT-XL/2-shaped 512^2 (or, with --res 256, 256^2) model, 250 transitions, guidance, batch B: images per second for the two bounding
    acceptance regimes (u = 0: every draft accepted; u = 1: a draft is accepted only if its log-ratio is >= 0, which a
    random-init drafter almost never reaches), for seeded uniforms, and for the plain sequential sampler (K = 0) on
    the same GPU.  One trajectory per regime after one warm-up trajectory; device time by CUDA events."""
    import json
    import torch
    import synth
    import paper_2511_20390_b200 as free
    torch.cuda.set_device(0)
    res = getattr(args, "res", 512)
    sh = synth.DIT_XL2_256 if res == 256 else synth.DIT_XL2_512
    B = args.batch or 16
    model = free.Model.random(sh, 1234, dtype="bf16", with_drafter=True)
    regimes = {"all_accepted": (K_DRAFTS, 0.0), "almost_all_rejected": (K_DRAFTS, 1.0),
               "seeded_uniforms": (K_DRAFTS, "seeded"), "sequential_K0": (0, None)}
    out = time_trajectories(model, sh, B, regimes, use_graph=getattr(args, "graph", False))
    line = {"metric": "images/s", "value": out["all_accepted"]["images_per_s"], "unit": "images/s", "n_gpus": 1,
            "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"sample_trajectory, DiT-XL/2-shaped {res}^2, {N_SCHED} transitions, K={K_DRAFTS}, cfg {CFG}, batch {B}"
                                   f"{', rounds replayed as a CUDA graph' if getattr(args, 'graph', False) else ''}; "
                                   "value = the all-accepted regime"},
            "regimes": out}
    print(json.dumps(line))
