#!/usr/bin/env python
"""Benchmark of the fused causal attention path (forward + backward preprocess + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
    python bench.py --workload long_context --profile --steps 1 --warmup 1     (a short run to put under ncu)
    python bench.py --grid causal|noncausal|fused|deterministic                (the paper's shape ranges)

One step = nova_attn_fwd + nova_attn_bwd_preprocess + nova_attn_bwd over one batch of the GPT-2-small
training attention shape (B=8, H=12, T=1024, D=64, causal, bf16).  Prints ONE JSON line.

  value      counted causal TFLOP/s (fwd 2*B*H*T^2*D, bwd 2.5x) of the whole job, inputs resident in
             HBM, timed with CUDA events on the launching stream, max over ranks.
  e2e        the same metric with the step's inputs copied from pinned host memory and its results
             copied back inside the timed region.
  roofline   tensor-core roofline of the dominant kernel (the fused backward) against the measured burst
             bf16 peak, from a second pass that brackets each kernel with events, and the forward and the
             whole backward (preprocess + clear + main + convert, timed in sequence) against the targets of
             50 % and 35 % of that peak.
  cpu_baseline  the fp64 oracle timed on the host cores on a bounded sample of the same workload.

With N > 1 (launched by torchrun, one rank per GPU) every rank runs the same per-GPU batch on its own
data: weak scaling, no data-path collective.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import functools
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2608_00029_b200 import multi, workloads as W  # noqa: E402

METRIC = "causal_attn_fwd_bwd_tflops"
UNIT = "TFLOP/s"
WORKLOAD = "gpt2_small"
L2_BYTES = 126e6
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler(threading.Thread):
    """Samples SM clock, power and clock-event reasons through NVML (read-only) while the GPU works."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, device_index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []  # (t, sm_mhz, reasons_mask, power_w)
        self._halt = threading.Event()
        self.ok = False
        self.max_mhz = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self._halt.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                try:
                    pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    pw = None
                self.samples.append((time.perf_counter(), mhz, mask, pw))
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self):
        self._halt.set()

    def summary(self, t0: float, t1: float) -> dict:
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "note": "NVML unavailable"}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = "sampled during the timed region"
        if len(inside) < 3:
            busy = sorted(self.samples, key=lambda s: -(s[3] or 0))[: max(3, len(self.samples) // 4)]
            inside = busy
            note = "timed region shorter than the sampling period: highest-power samples of the whole run"
        clocks = sorted(s[1] for s in inside)
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [name for bit, name in self.REASONS.items() if mask & bit]
        powers = [s[3] for s in inside if s[3] is not None]
        return {"sm_mhz": clocks[len(clocks) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "power_w_max": max(powers) if powers else None, "note": note}


# ------------------------------------------------------------------------------------------ oracle leg
def time_oracle(cfg, Q, K, V, dO, budget_s: float = 12.0, max_batches: int | None = None):
    """Times the fp64 CPU oracle (forward + backward) batch by batch until about `budget_s` seconds of
    work are done.  Returns (TFLOP/s, threads, description of the sample)."""
    import oracle
    threads = oracle.num_threads()
    per_batch_flops = (cfg.fwd_flops + cfg.bwd_flops) / cfg.B
    done, spent = 0, 0.0
    nb = cfg.B if max_batches is None else min(cfg.B, max_batches)
    for b in range(nb):
        q, k, v, do = (W.widen(x[b:b + 1]) for x in (Q, K, V, dO))
        t0 = time.perf_counter()
        oracle.attn_fwd(q, k, v, cfg.scale, cfg.causal)
        oracle.attn_bwd(q, k, v, do, cfg.scale, cfg.causal)
        spent += time.perf_counter() - t0
        done += 1
        if spent >= budget_s:
            break
    tflops = done * per_batch_flops / spent / 1e12
    sample = f"{done} of {cfg.B} sequences ({done * cfg.H} heads) of {cfg.name}, fwd+bwd once, {spent:.2f} s"
    return tflops, threads, sample, spent / done


def run_reference(args):
    """The reference arm of this build is the fp64 CPU oracle as it stands.  Each step runs it forward +
    backward on a bounded sample of the workload: one whole sequence (all heads of one batch entry)
    when K + W such steps fit in about four minutes, otherwise a single head."""
    rank, _, world = multi.env_rank_world()
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    cfg = W.CONFIGS[args.workload]
    Q, K, V, dO = W.make_inputs(cfg)
    threads = oracle.num_threads()

    def run_sample(b, heads):
        q, k, v, do = (W.widen(x[b:b + 1, :heads]) for x in (Q, K, V, dO))
        oracle.attn_fwd(q, k, v, cfg.scale, cfg.causal)
        oracle.attn_bwd(q, k, v, do, cfg.scale, cfg.causal)

    t0 = time.perf_counter()
    run_sample(0, cfg.H)  # calibration, untimed
    t_seq = time.perf_counter() - t0
    heads = cfg.H if t_seq * (args.steps + args.warmup) <= 240.0 else 1
    for i in range(args.warmup):
        run_sample(i % cfg.B, heads)
    t0 = time.perf_counter()
    for i in range(args.steps):
        run_sample(i % cfg.B, heads)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    flops = (cfg.fwd_flops + cfg.bwd_flops) / (cfg.B * cfg.H) * heads
    value = flops / dt / 1e12
    sample = f"{heads} of {cfg.B * cfg.H} heads of {cfg.name} per step, fwd+bwd"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "T": cfg.T, "D": cfg.D, "causal": True,
                   "note": "fp64 CPU oracle on the host cores; each step is a bounded sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(threads, heads), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------ our arm
class BufferSet:
    def __init__(self, cfg, dev, inputs):
        from paper_2608_00029_b200 import nova_attn
        self.q, self.k, self.v, self.do = (x.to(dev) for x in inputs)
        shape = (cfg.B, cfg.H, cfg.T, cfg.D)
        self.o, self.dq, self.dk, self.dv = (torch.empty(shape, dtype=torch.bfloat16, device=dev) for _ in range(4))
        self.lse = torch.empty((cfg.B, cfg.H, cfg.T), dtype=torch.float32, device=dev)
        self.delta = torch.empty_like(self.lse)
        self.ws = torch.empty(nova_attn.nova_attn_bwd_workspace_bytes(*shape), dtype=torch.uint8, device=dev)

    def bytes(self):
        t = (self.q, self.k, self.v, self.do, self.o, self.dq, self.dk, self.dv, self.lse, self.delta, self.ws)
        return sum(x.numel() * x.element_size() for x in t)


def step(na, cfg, s):
    na.nova_attn_fwd(s.q, s.k, s.v, s.o, s.lse, cfg.scale, cfg.causal)
    na.nova_attn_bwd_preprocess(s.o, s.do, s.delta)
    na.nova_attn_bwd(s.q, s.k, s.v, s.o, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, cfg.causal, s.ws)


def run_profile(args, na, cfg, dev):
    """A short run of the step on one buffer set, nothing else: the command to put under a profiler."""
    s = BufferSet(cfg, dev, W.make_inputs(cfg))
    for _ in range(args.warmup + args.steps):
        step(na, cfg, s)
    na.nova_attn_poll_device_status()
    print(json.dumps({"profile_run": cfg.name, "B": cfg.B, "H": cfg.H, "T": cfg.T, "D": cfg.D,
                      "steps": args.warmup + args.steps, "checksum": float(s.dq.float().sum())}), flush=True)
    return 0


# The eight shapes of the grid lie inside the ranges of the paper's attention microbenchmark (Section 6.1:
# sequence lengths 512 to 2048, 12 to 32 heads, head dimension 64 or 128; the per-shape values are in a
# figure), at batch 16 like that figure's "16x12x64" label.
GRID = [(512, 12, 64), (1024, 12, 64), (2048, 12, 64), (1024, 16, 64), (1024, 20, 64), (512, 32, 128),
        (1024, 32, 128), (2048, 32, 128)]  # (T, H, D)


class GridSet:
    """One set of buffers for a grid shape, plain [B,H,T,D] or the fused-projection layout (Q, K, V read in
    place from [B,T,3,H,D], O / dO as [B,T,H,D], dQ, dK, dV written into one [B,T,3,H,D] buffer)."""

    def __init__(self, na, cfg, dev, inputs, fused):
        B, H, T, D = cfg.B, cfg.H, cfg.T, cfg.D
        q, k, v, do = (x.to(dev) for x in inputs)
        self.lse = torch.empty((B, H, T), dtype=torch.float32, device=dev)
        self.delta = torch.empty_like(self.lse)
        self.ws = torch.empty(na.nova_attn_bwd_workspace_bytes(B, H, T, D), dtype=torch.uint8, device=dev)
        if fused:
            qkv = torch.empty((B, T, 3, H, D), dtype=torch.bfloat16, device=dev)
            for i, x in enumerate((q, k, v)):
                qkv[:, :, i] = x.permute(0, 2, 1, 3)
            dqkv = torch.empty_like(qkv)
            self.keep = (qkv, dqkv)
            self.q, self.k, self.v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
            self.dq, self.dk, self.dv = (dqkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
            self.o = torch.empty((B, T, H, D), dtype=torch.bfloat16, device=dev).permute(0, 2, 1, 3)
            self.do = do.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        else:
            self.q, self.k, self.v, self.do = q, k, v, do
            self.o, self.dq, self.dk, self.dv = (torch.empty_like(q) for _ in range(4))
        self.nbytes = 8 * q.numel() * 2 + 2 * self.lse.numel() * 4 + self.ws.numel()


def run_grid(args):
    """Forward and backward (preprocess + backward) timed over the grid through the same protocol as the
    headline number: buffer sets in rotation so that no call finds its inputs in L2, warm-up, CUDA events
    on the launching stream around `--steps` calls issued one by one, clocks sampled meanwhile.  Prints a
    markdown table and one JSON line with the rows and the clock record."""
    from paper_2608_00029_b200 import nova_attn as na
    na.load()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream()
    mode = args.grid
    causal = mode != "noncausal"
    fused, det = mode == "fused", mode == "deterministic"
    sampler = ClockSampler(0)
    sampler.start()
    t_region0 = time.perf_counter()
    rows = []
    print("| B | H | T | D | causal | fwd ms | fwd TFLOP/s | bwd ms | bwd TFLOP/s | fwd+bwd ms |", file=sys.stderr)
    print("|---|---|---|---|---|---|---|---|---|---|", file=sys.stderr)
    for T, H, D in GRID:
        cfg = W.AttnConfig(f"grid_T{T}_H{H}_D{D}", B=args.grid_batch, H=H, T=T, D=D, seed=5, causal=causal)
        first = GridSet(na, cfg, dev, W.make_inputs(cfg), fused)
        n_sets = max(2, int(L2_BYTES * 2 // first.nbytes) + 2)
        sets = [first] + [GridSet(na, cfg, dev, W.make_inputs(cfg, seed=5 + i), fused) for i in range(1, n_sets)]

        def fwd(s):
            if fused:
                na.nova_attn_fwd_strided(s.q, s.k, s.v, s.o, s.lse, cfg.scale, causal)
            else:
                na.nova_attn_fwd(s.q, s.k, s.v, s.o, s.lse, cfg.scale, causal)

        def bwd(s):
            if fused:
                na.nova_attn_bwd_preprocess_strided(s.o, s.do, s.delta)
                na.nova_attn_bwd_strided(s.q, s.k, s.v, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, causal, s.ws)
                return
            na.nova_attn_bwd_preprocess(s.o, s.do, s.delta)
            if det:
                na.nova_attn_bwd_deterministic(s.q, s.k, s.v, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, causal)
            else:
                na.nova_attn_bwd(s.q, s.k, s.v, s.o, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, causal, s.ws)

        def timed(fn):
            for i in range(max(args.warmup, 3)):
                fn(sets[i % n_sets])
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(args.steps):
                fn(sets[i % n_sets])
            e1.record(stream)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        for s in sets:  # every set holds a valid O, LSE, Delta before the backward is timed
            fwd(s)
        t_f, t_b = timed(fwd), timed(bwd)
        na.nova_attn_poll_device_status()
        f_flops = cfg.fwd_flops * (1.0 if causal else 2.0)  # the counted figure covers half the square
        row = {"B": cfg.B, "H": H, "T": T, "D": D, "causal": causal, "fwd_ms": t_f, "fwd_tflops": f_flops / t_f / 1e9,
               "bwd_ms": t_b, "bwd_tflops": 2.5 * f_flops / t_b / 1e9, "buffer_sets": n_sets}
        rows.append(row)
        print(f"| {cfg.B} | {H} | {T} | {D} | {'yes' if causal else 'no'} | {t_f:.4f} | {row['fwd_tflops']:.0f} | "
              f"{t_b:.4f} | {row['bwd_tflops']:.0f} | {t_f + t_b:.4f} |", file=sys.stderr, flush=True)
        del sets, first
        torch.cuda.empty_cache()
    sampler.stop()
    sampler.join(timeout=2)
    print(json.dumps({"grid": mode, "steps": args.steps, "warmup": max(args.warmup, 3), "launch": "eager",
                      "l2": "buffer sets in rotation, more than twice the 126 MB L2 between two uses of a set",
                      "rows": rows, "clocks": sampler.summary(t_region0, time.perf_counter())}), flush=True)
    return 0


def run_lmhead(args):
    """The second workload: the fused loss head (projection + softmax cross-entropy statistics + merge) on the
    paper's shape.  One step = one nova_lmhead_fwd call; value = projection TFLOP/s (2*M*N*K)."""
    from paper_2608_00029_b200 import nova_attn as na, nova_lmhead as lm
    na.load()
    rank, local_rank, world = multi.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the loss head has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        multi.init_process_group("nccl")
    peaks, peak_src = load_peaks()
    cfg = W.LM_HEAD_CONFIGS[args.workload]  # rows are independent: every rank runs the same number of rows
    stream = torch.cuda.current_stream()

    def make_set(seed):
        X, Wm, t = (a.to(dev) for a in W.make_lmhead_inputs(cfg, seed=seed))
        return {"X": X, "W": Wm, "t": t, "logits": torch.empty((cfg.M, cfg.N), dtype=torch.bfloat16, device=dev),
                "lse": torch.empty(cfg.M, dtype=torch.float32, device=dev),
                "loss": torch.empty(cfg.M, dtype=torch.float32, device=dev),
                "ws": torch.empty(lm.nova_lmhead_workspace_bytes(cfg.M, cfg.N, cfg.K), dtype=torch.uint8, device=dev)}

    sets = [make_set(cfg.seed + 1000 * rank + i) for i in range(2)]  # each set (logits alone 0.8 GB) exceeds L2
    set_bytes = sum(v.numel() * v.element_size() for v in sets[0].values())

    def step(s):
        lm.nova_lmhead_fwd(s["X"], s["W"], s["t"], s["logits"], s["lse"], s["loss"], s["ws"])

    if args.profile:
        for i in range(args.warmup + args.steps):
            step(sets[0])
        na.nova_attn_poll_device_status()
        print(json.dumps({"profile_run": cfg.name, "M": cfg.M, "N": cfg.N, "K": cfg.K, "steps": args.warmup + args.steps,
                          "checksum": float(sets[0]["loss"].sum())}), flush=True)
        return 0

    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(sets[i % 2])
    torch.cuda.synchronize()
    multi.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ev0.record(stream)
    for i in range(args.steps):
        step(sets[i % 2])
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    multi.barrier()
    ms = multi.max_over_ranks(ev0.elapsed_time(ev1), dev) / args.steps
    na.nova_attn_poll_device_status()
    value = cfg.flops * world / (ms * 1e-3) / 1e12

    # the contraction kernel alone (it is followed at once by the merge: time the pair, then the pair without
    # the logits, which removes the only large store)
    def timed(fn, n):
        for i in range(3):
            fn(sets[i % 2])
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(n):
            fn(sets[i % 2])
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n

    n_attr = min(args.steps, 50)
    ms_nolog = timed(lambda s: lm.nova_lmhead_fwd(s["X"], s["W"], s["t"], None, s["lse"], s["loss"], s["ws"]), n_attr)

    # context only: the same chain as three library calls (projection, log-softmax pass, NLL pick)
    def library_chain(s):
        z = torch.matmul(s["X"], s["W"].T, out=s["logits"])
        return torch.logsumexp(z, dim=1)

    try:
        ms_lib_gemm = timed(lambda s: torch.matmul(s["X"], s["W"].T, out=s["logits"]), n_attr)
        ms_lib_chain = timed(library_chain, n_attr)
    except Exception:
        ms_lib_gemm = ms_lib_chain = None

    # end to end: the step's hidden states and targets come from pinned host memory, its losses go back
    hX = [sets[i]["X"].cpu().pin_memory() for i in range(2)]
    hT = [sets[i]["t"].cpu().pin_memory() for i in range(2)]
    hOut = [torch.empty((2, cfg.M), dtype=torch.float32).pin_memory() for _ in range(2)]

    def e2e_step(i):
        s = sets[i % 2]
        s["X"].copy_(hX[i % 2], non_blocking=True)
        s["t"].copy_(hT[i % 2], non_blocking=True)
        step(s)
        hOut[i % 2][0].copy_(s["lse"], non_blocking=True)
        hOut[i % 2][1].copy_(s["loss"], non_blocking=True)

    n_e2e = max(3, min(args.steps, 50))
    for i in range(3):
        e2e_step(i)
    torch.cuda.synchronize()
    multi.barrier()
    ev0.record(stream)
    for i in range(n_e2e):
        e2e_step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    multi.barrier()
    e2e_ms = multi.max_over_ranks(ev0.elapsed_time(ev1), dev) / n_e2e
    sampler.stop()
    sampler.join(timeout=2)

    cpu_baseline = None
    if rank == 0 and world == 1:
        import oracle
        oracle.build()
        X, Wm, t = W.make_lmhead_inputs(cfg)
        Wd = W.widen(Wm)
        rows, spent = 0, 0.0
        chunk = 48
        while spent < 10.0 and rows < cfg.M:
            tt = time.perf_counter()
            oracle.lmhead_fwd(W.widen(X[rows:rows + chunk]), Wd, t[rows:rows + chunk].numpy())
            spent += time.perf_counter() - tt
            rows += chunk
        cpu_baseline = {"value": 2.0 * rows * cfg.N * cfg.K / spent / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
                        "kind": "oracle", "sample": f"{rows} of {cfg.M} rows of {cfg.name}, {spent:.2f} s"}

    if rank == 0:
        peak = peaks["bf16_tflops"]
        ach = cfg.flops / (ms * 1e-3) / 1e12
        # DRAM bytes of one launch of the main kernel from the committed ncu summary of this very workload
        traffic, traffic_source = None, None
        traffic_rel = os.path.join("profiles", f"lmhead_pair_kernel_{cfg.name}.md")
        if os.path.exists(os.path.join(ROOT, traffic_rel)):
            with open(os.path.join(ROOT, traffic_rel)) as f:
                for ln in f:
                    if ln.startswith("traffic_bytes_per_launch:"):
                        traffic = int(ln.split(":")[1])
                        traffic_source = f"{traffic_rel} (committed ncu summary, not measured in this run)"
        line = {
            "metric": "lm_head_fused_tflops", "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": cfg.name, "M": cfg.M, "N": cfg.N, "K": cfg.K, "logits": "bf16, stored",
                       "parallelism": f"dp{world} (rows split, no collective)",
                       "l2": f"alternating 2 buffer sets of {set_bytes / 1e6:.0f} MB (> 126 MB L2)",
                       "launch": "eager (2 kernels per step)",
                       "context": "the paper's fused loss head takes 7.91 ms on an RTX 6000 Ada (TF32, fp32 logits)"},
            "e2e": {"value": cfg.flops * world / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": int(hX[0].numel() * 2 + hT[0].numel() * 4), "d2h_bytes_per_step": int(cfg.M * 8),
                    "ms_per_step": e2e_ms, "steps": n_e2e},
            "gpu_launches": 2 * args.steps,
            "clocks": sampler.summary(t0, t1),
            "roofline": {"bound": "tensor", "kernel": "lmhead_pair_kernel (+ lmhead_merge_kernel)", "achieved": ach,
                         "peak": peak, "unit": UNIT, "frac": ach / peak, "traffic": traffic, "traffic_source": traffic_source,
                         "peak_source": f"{peak_src} bf16_tflops (burst)",
                         "ms_per_launch": ms, "ms_without_logits": ms_nolog,
                         "library_context": {"what": "torch.matmul alone / torch.matmul + logsumexp over the stored logits",
                                             "ms_gemm": ms_lib_gemm, "ms_gemm_plus_reduction": ms_lib_chain}},
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        multi.barrier()
        torch.distributed.destroy_process_group()
    return 0


def run_ours(args):
    from paper_2608_00029_b200 import nova_attn as na
    na.load()  # fails loudly if the CUDA library has not been built
    rank, local_rank, world = multi.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        multi.init_process_group("nccl")
    peaks, peak_src = load_peaks()

    base = W.CONFIGS[args.workload]
    plan = multi.weak_scaling_plan(base.B, world, rank)
    cfg = base.replace(B=plan["local_batch"])
    if args.profile:
        return run_profile(args, na, cfg, dev)
    # Rotate over enough independent buffer sets that the data touched between two uses of the same
    # set exceeds L2, so no step finds its inputs cached from the previous use.
    probe = BufferSet(cfg, dev, W.make_inputs(cfg, seed=base.seed + 1000 * rank))
    n_sets = max(2, int(L2_BYTES * 2 // probe.bytes()) + 2)
    sets = [probe] + [BufferSet(cfg, dev, W.make_inputs(cfg, seed=base.seed + 1000 * rank + i)) for i in range(1, n_sets)]
    stream = torch.cuda.current_stream()
    flops_step = cfg.fwd_flops + cfg.bwd_flops

    sampler = ClockSampler(local_rank)
    sampler.start()

    # ---- device-resident timing
    # One step's five launches (the same C-ABI calls) are recorded once per buffer set into a CUDA graph
    # and replayed, as a training loop that has captured its step would run them; --launch eager issues
    # the calls one by one instead.
    run_step = [functools.partial(step, na, cfg, s) for s in sets]
    launch_mode = args.launch
    eager_step = run_step

    def run_round():
        for f in eager_step:
            f()

    if launch_mode == "graph":
        cap = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(cap):
            run_round()
        cap.synchronize()
        try:
            # thread_local: CUDA calls of other threads (a process group's watchdog) do not end the capture
            graphs = []
            for s in sets:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=cap, capture_error_mode="thread_local"):
                    step(na, cfg, s)
                graphs.append(g)
            # one round over all buffer sets as a single graph: the steps inside keep their programmatic
            # dependent launch across step boundaries
            g_round = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_round, stream=cap, capture_error_mode="thread_local"):
                for s in sets:
                    step(na, cfg, s)
            run_step = [g.replay for g in graphs]
            run_round = g_round.replay
        except Exception as e:  # the eager calls are the same work: fall back and say so
            print(f"bench.py: CUDA graph capture failed ({e!r}); timing eager launches", file=sys.stderr)
            torch.cuda.synchronize()
            launch_mode = "eager"

    def run_steps(n):  # exactly n steps, buffer sets in rotation
        for _ in range(n // n_sets):
            run_round()
        for i in range(n % n_sets):
            run_step[i]()

    run_steps(max(args.warmup, 3))
    torch.cuda.synchronize()
    multi.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t_region0 = time.perf_counter()
    ev0.record(stream)
    run_steps(args.steps)
    ev1.record(stream)
    torch.cuda.synchronize()
    t_region1 = time.perf_counter()
    multi.barrier()
    ms_total = multi.max_over_ranks(ev0.elapsed_time(ev1), dev)
    na.nova_attn_poll_device_status()
    ms_per_step = ms_total / args.steps
    value = flops_step * world / (ms_per_step * 1e-3) / 1e12

    # ---- per-kernel attribution.  Two passes over the same rotation of buffer sets:
    # (1) each kernel's launches recorded back to back into a CUDA graph and replayed, as they run inside the
    #     timed steps (no host in between): `kernel_ms`, the figure the roofline uses;
    # (2) the calls issued one by one with an event on either side: `kernel_ms_eager`.  The host needs longer to
    #     issue a launch and two event records than these kernels run, so this figure contains idle time.
    names = ["fwd", "bwd_preprocess", "bwd_zero", "bwd_main", "bwd_convert"]

    def one_kernel(name, s):
        if name == "fwd":
            na.nova_attn_fwd(s.q, s.k, s.v, s.o, s.lse, cfg.scale, cfg.causal)
        elif name == "bwd_preprocess":
            na.nova_attn_bwd_preprocess(s.o, s.do, s.delta)
        elif name == "bwd":  # the whole backward as the three calls make it: preprocess + clear + main + convert
            na.nova_attn_bwd_preprocess(s.o, s.do, s.delta)
            na.nova_attn_bwd(s.q, s.k, s.v, s.o, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, cfg.causal, s.ws)
        else:
            bit = {"bwd_zero": na.BWD_STEP_ZERO, "bwd_main": na.BWD_STEP_MAIN, "bwd_convert": na.BWD_STEP_CONVERT}[name]
            na.nova_attn_bwd(s.q, s.k, s.v, s.o, s.do, s.lse, s.delta, s.dq, s.dk, s.dv, cfg.scale, cfg.causal, s.ws,
                             steps=bit)

    def graph_ms(name, rounds=8, reps=5):
        """Mean duration of `name`, launched rounds * n_sets times back to back from a CUDA graph."""
        side = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            for s in sets:
                one_kernel(name, s)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
            for _ in range(rounds):
                for s in sets:
                    one_kernel(name, s)
        g.replay()
        torch.cuda.synchronize()
        times = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b) / (rounds * n_sets))
        return sorted(times)[len(times) // 2]

    attribution = "CUDA graph of back-to-back launches per kernel"
    try:
        kernel_ms = {n: graph_ms(n) for n in names}
        fwd_seq_ms, bwd_seq_ms = kernel_ms["fwd"], graph_ms("bwd")
    except Exception as e:  # capture unavailable: fall back to the eager figures and say so
        print(f"bench.py: per-kernel graph capture failed ({e!r}); using eager launches", file=sys.stderr)
        torch.cuda.synchronize()
        kernel_ms = None
        attribution = "eager launches between events (contains host gaps)"

    k_steps = min(args.steps, 200)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)] for _ in range(k_steps)]
    for i in range(k_steps):
        s = sets[i % n_sets]
        e = evs[i]
        e[0].record(stream)
        for j, n in enumerate(names):
            one_kernel(n, s)
            e[j + 1].record(stream)
    torch.cuda.synchronize()
    kernel_ms_eager = {n: sum(e[i].elapsed_time(e[i + 1]) for e in evs) / k_steps for i, n in enumerate(names)}
    if kernel_ms is None:
        kernel_ms = kernel_ms_eager
        fwd_seq_ms = kernel_ms["fwd"]
        bwd_seq_ms = sum(kernel_ms[n] for n in names[1:])

    bwd_ms = kernel_ms["bwd_main"]
    achieved = cfg.bwd_flops / (bwd_ms * 1e-3) / 1e12
    # these passes are a few milliseconds of work at full clocks: the burst figure is the peak that applies;
    # the sustained one is given beside it
    peak = peaks["bf16_tflops"]
    fwd_tflops = cfg.fwd_flops / (fwd_seq_ms * 1e-3) / 1e12
    bwd_tflops = cfg.bwd_flops / (bwd_seq_ms * 1e-3) / 1e12
    roofline = {
        "bound": "tensor", "kernel": "attn_bwd_kernel", "achieved": achieved, "peak": peak, "unit": UNIT,
        "frac": achieved / peak, "traffic": None, "traffic_source": None,
        "peak_source": f"{peak_src} bf16_tflops (burst)",
        "peak_sustained": peaks["bf16_tflops_sustained"],
        "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"], "ms_per_launch": bwd_ms,
        "kernel_ms": kernel_ms, "kernel_ms_eager": kernel_ms_eager, "attribution": attribution,
        "targets": {
            "fwd": {"what": "nova_attn_fwd", "ms": fwd_seq_ms, "tflops": fwd_tflops, "frac": fwd_tflops / peak,
                    "target": 0.50},
            "bwd": {"what": "nova_attn_bwd_preprocess + nova_attn_bwd (clear, main, convert) in sequence",
                    "ms": bwd_seq_ms, "tflops": bwd_tflops, "frac": bwd_tflops / peak, "target": 0.35},
        },
        "preprocess_gbs": (4.0 * cfg.B * cfg.H * cfg.T * cfg.D + 4.0 * cfg.B * cfg.H * cfg.T)
        / (kernel_ms["bwd_preprocess"] * 1e-3) / 1e9,
        "preprocess_frac_of_hbm_peak": (4.0 * cfg.B * cfg.H * cfg.T * cfg.D + 4.0 * cfg.B * cfg.H * cfg.T)
        / (kernel_ms["bwd_preprocess"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
    }
    # DRAM bytes of one launch of the dominant kernel are not measured by this run: they come from the
    # committed ncu summary of this workload (its "traffic_bytes_per_launch: N" line); absent or another
    # workload -> null.
    traffic_rel = os.path.join("profiles", f"attn_bwd_kernel_{base.name}.md")
    traffic_path = os.path.join(ROOT, traffic_rel)
    if os.path.exists(traffic_path) and cfg.B == base.B:
        try:
            with open(traffic_path) as f:
                for line in f:
                    if line.startswith("traffic_bytes_per_launch:"):
                        roofline["traffic"] = int(line.split(":")[1])
                        roofline["traffic_source"] = f"{traffic_rel} (committed ncu summary, not measured in this run)"
        except Exception:
            pass

    # ---- end to end: pinned host inputs in, results out, every step
    host_in = [tuple(x.pin_memory() for x in W.make_inputs(cfg, seed=base.seed + 1000 * rank + 7)) for _ in range(2)]
    host_out = [tuple(torch.empty((cfg.B, cfg.H, cfg.T, cfg.D), dtype=torch.bfloat16).pin_memory() for _ in range(4))
                for _ in range(2)]
    h2d = sum(x.numel() * x.element_size() for x in host_in[0])
    d2h = sum(x.numel() * x.element_size() for x in host_out[0])

    # Three streams, as a caller that feeds the library from the host would run it: the copies of step
    # i+1's inputs and of step i-1's results overlap step i's kernels (PCIe is full duplex).  Every step
    # still moves all of its inputs in and all of its results out inside the timed region.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    set_free = [None] * n_sets  # event: the results of the last step that used the set have left the device

    def e2e_step(i):
        k = i % n_sets
        s = sets[k]
        hi, ho = host_in[i % 2], host_out[i % 2]
        with torch.cuda.stream(s_in):
            if set_free[k] is not None:
                s_in.wait_event(set_free[k])
            for dst, src in zip((s.q, s.k, s.v, s.do), hi):
                dst.copy_(src, non_blocking=True)
            in_ready = s_in.record_event()
        stream.wait_event(in_ready)
        step(na, cfg, s)
        done = stream.record_event()
        with torch.cuda.stream(s_out):
            s_out.wait_event(done)
            for dst, src in zip(ho, (s.o, s.dq, s.dk, s.dv)):
                dst.copy_(src, non_blocking=True)
            set_free[k] = s_out.record_event()

    def e2e_join():  # the launching stream waits for the copies still in flight
        for e in set_free:
            if e is not None:
                stream.wait_event(e)

    e2e_steps = max(3, min(args.steps, 50))
    for i in range(3):
        e2e_step(i)
    e2e_join()
    torch.cuda.synchronize()
    multi.barrier()
    ev0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    e2e_join()
    ev1.record(stream)
    torch.cuda.synchronize()
    multi.barrier()
    e2e_ms = multi.max_over_ranks(ev0.elapsed_time(ev1), dev) / e2e_steps
    e2e_value = flops_step * world / (e2e_ms * 1e-3) / 1e12
    na.nova_attn_poll_device_status()

    sampler.stop()
    sampler.join(timeout=2)
    clocks = sampler.summary(t_region0, t_region1)

    cpu_baseline = None
    if rank == 0 and world == 1:
        import oracle
        oracle.build()
        inputs = W.make_inputs(base)
        v, threads, sample, _ = time_oracle(base, *inputs, budget_s=12.0)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": min(threads, base.H), "kind": "oracle", "sample": sample}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": base.name, "B_per_gpu": cfg.B, "global_batch": plan["global_batch"], "H": cfg.H,
                       "T": cfg.T, "D": cfg.D, "causal": True, "parallelism": f"dp{world} (batch split, no collective)",
                       "l2": f"rotating {n_sets} buffer sets of {probe.bytes() / 1e6:.0f} MB "
                             f"({n_sets * probe.bytes() / 1e6:.0f} MB > 126 MB L2)",
                       "launch": (f"CUDA graph of one round over the {n_sets} buffer sets, replayed (5 kernels per step)"
                                  if launch_mode == "graph" else "eager (5 launches per step)"),
                       "flops_per_step": flops_step, "frac_of_burst_peak": value / world / peaks["bf16_tflops"]},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "steps": e2e_steps},
            "gpu_launches": 5 * args.steps,
            "clocks": clocks,
            "roofline": roofline,
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        multi.barrier()
        torch.distributed.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--launch", choices=["graph", "eager"], default="graph",
                    help="timed steps replayed from a CUDA graph per buffer set (default) or issued call by call")
    ap.add_argument("--workload", choices=W.CONFIG_ORDER + sorted(W.LM_HEAD_CONFIGS), default=WORKLOAD,
                    help="the configuration to run (the headline number is quoted on the default)")
    ap.add_argument("--profile", action="store_true",
                    help="only run warmup + steps steps on one buffer set and exit: a short command for a profiler")
    ap.add_argument("--grid", choices=["causal", "noncausal", "fused", "deterministic"], default=None,
                    help="time forward and backward over the paper's shape ranges instead of the headline workload")
    ap.add_argument("--grid-batch", type=int, default=16)
    args = ap.parse_args()
    if args.grid:
        if args.steps == 500:
            args.steps = 30
        return run_grid(args)
    if args.workload in W.LM_HEAD_CONFIGS:
        if args.impl == "reference":
            raise SystemExit("--impl reference times the attention oracle: use an attention workload")
        if args.steps == 500:
            args.steps = 100
        return run_lmhead(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
