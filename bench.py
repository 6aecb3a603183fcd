#!/usr/bin/env python
"""Benchmark of the fused MoE forward (EP=1) on the Mixtral-like layer (T=8192, H=4096, F=14336, E=8, top-2).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--impl reference] [--sweep]

A step is one pass of the whole hot path (routing plan, dispatch, Linear-1 + SiLU*mul, Linear-2,
combine) over one batch of seeded synthetic tokens.  The reported value is the steady-state one: the timed steps
run back to back after at least two seconds of pre-heating steps, when the power cap has settled the clocks; the
figure of the first steps after the warm-up is kept beside it (burst_*).  With N > 1 (torchrun) every rank runs the same
layer on its own batch (experts replicated, tokens data-parallel, no collective on the data path):
weak scaling; the reported value is all ranks' tokens over the slowest rank's device time.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2607_23264_b200 import inputs as gen  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

def dram_traffic_per_expert(kernel: str, H: int, F: int):
    """ncu DRAM bytes (read + write) of one Linear-1 launch, per non-empty expert, for `kernel` on experts of shape
    H x F, from the committed summary of the captures (a table row per kernel and expert shape: name | case |
    experts | dram read bytes | dram write bytes; the case names its "H=..., F=...").  None when the summary or the
    row is missing."""
    path = os.path.join(ROOT, "profiles", "linear1_dram_traffic.md")
    try:
        with open(path) as fh:
            for line in fh:
                cells = [c.strip() for c in line.strip().strip("|").split("|")]
                if len(cells) >= 5 and cells[0].strip("`") == kernel and f"H={H}, F={F}" in cells[1]:
                    experts, rd, wr = int(cells[2]), int(cells[3].replace(",", "")), int(cells[4].replace(",", ""))
                    return (rd + wr) / experts
    except (OSError, ValueError):
        pass
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap,temperature.gpu")

    def __init__(self, index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, power, temp, reasons = [], [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            try:
                temp.append(float(parts[7]))      # context: a hotter die leaks more and holds a lower clock at the cap
            except (ValueError, IndexError):
                pass
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        busy = [v for v in sm if v > 0]
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "power_w_median": statistics.median(power) if power else None, "power_w_max": max(power) if power else None,
                "temp_c_median": statistics.median(temp) if temp else None}


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_rate(cfg, x_bits, logits, weights, n_tokens, seed=1234):
    """Time the CPU oracle on a seeded sample of tokens of this workload.  Returns (tokens/s, seconds)."""
    from oracle import moe_oracle as orc
    rng = np.random.default_rng(seed)
    toks = np.sort(rng.choice(cfg.T, size=min(n_tokens, cfg.T), replace=False))
    t0 = time.perf_counter()
    orc.forward_tokens(toks, x_bits, logits, cfg.k, weights)
    dt = time.perf_counter() - t0
    return len(toks) / dt, dt


def run_reference(args, cfg, rank, world):
    """--impl reference: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    x_bits = gen.make_x(cfg)
    logits = gen.make_logits(cfg, x_bits)
    W = gen.stacked_weights(cfg)
    weights = lambda e: (W[0][e], W[1][e], W[2][e])
    n_tok = args.ref_tokens
    for _ in range(args.warmup):
        oracle_sample_rate(cfg, x_bits, logits, weights, n_tok)
    times = []
    for s in range(args.steps):
        _, dt = oracle_sample_rate(cfg, x_bits, logits, weights, n_tok, seed=1000 + s)
        times.append(dt)
    total = sum(times)
    value = n_tok * args.steps / total
    cores = oracle_threads()
    sample = (f"{n_tok} seeded-random tokens of {cfg.name} per step (row-sampled fp64 oracle, exact per row; the oracle's "
              "widening of each touched expert's bf16 matrices to fp64 is part of the timed call)")
    line = {
        "impl": "reference", "metric": "fused MoE fwd tokens/s", "value": value, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args.gpus),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(cfg, n_gpus):
    return {"workload": f"{cfg.name}: T={cfg.T} tokens per GPU, hidden={cfg.H}, ffn={cfg.F}, E={cfg.E}, top-{cfg.k}, "
                        f"SwiGLU, bf16, router={cfg.router}, seed={cfg.seed}",
            "tokens_per_gpu": cfg.T, "global_tokens": cfg.T * n_gpus, "parallelism": f"ep1 x {n_gpus} replicas",
            "l2_policy": "inputs larger than L2 (%.1f GB of weights + %.2f GB of activations per step vs 126 MB L2)"
                         % (6 * cfg.E * cfg.H * cfg.F / 1e9, (2 * cfg.T * cfg.H + 4 * cfg.R * cfg.H + 2 * cfg.R * cfg.F) * 2 / 1e9)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="C2", choices=sorted(gen.CONFIGS))
    ap.add_argument("--tokens", type=int, default=0, help="run --config's layer at this batch size instead of its own T")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--ref-tokens", type=int, default=128, help="tokens per step of the reference (oracle) arm")
    ap.add_argument("--cpu-baseline-tokens", type=int, default=128,
                    help="tokens of the cpu_baseline leg (the same sample size as a step of the reference arm)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-local-peak", action="store_true",
                    help="skip the context measurement of the library bf16 GEMM on this GPU (after all timed regions)")
    ap.add_argument("--heat-seconds", type=float, default=2.0,
                    help="back-to-back untimed steps before the timed region, until the power cap has settled the clocks")
    ap.add_argument("--burst", type=int, default=1)
    ap.add_argument("--mode", type=int, default=0)
    ap.add_argument("--ik", type=int, default=1)
    ap.add_argument("--schedule", type=int, default=0, help="0 Expert-Wave order, 1 interleaved order (Algorithm 1)")
    ap.add_argument("--lead", type=int, default=0, help="schedule 1: row lead D (0 = the anti-starvation knee)")
    ap.add_argument("--one-launch", action="store_true", help="schedule 0 as one launch with ready counters")
    ap.add_argument("--pairs", choices=["auto", "on", "off"], default="auto",
                    help="CTA-pair (cta_group::2) kernel: auto = for layers with many rows per expert")
    ap.add_argument("--sweep", action="store_true", help="store-pacing sweep (20 points) instead of the bench line")
    ap.add_argument("--probe-mma", action="store_true",
                    help="print SM clocks per tcgen05.mma for several tile shapes (tensor-pipe calibration) and exit")
    ap.add_argument("--fp8", action="store_true",
                    help="time the FP8 (E4M3, W8A8) variant of the layer instead (weights quantised on the GPU first)")
    ap.add_argument("--mxfp8", action="store_true",
                    help="the block-scaled FP8 variant of the experts (E4M3 elements, E8M0 scale per 32 elements along K)")
    ap.add_argument("--library-gemms", action="store_true",
                    help="context, not the product: the layer's two grouped GEMMs as one library bf16 GEMM call per "
                         "expert (torch.matmul on the seeded routing's row ranges; no SiLU, no routing, no movers), "
                         "pre-heated, on this GPU")
    ap.add_argument("--router", action="store_true",
                    help="time the router front end (logits + top-k in one kernel, then the plan) on --config's shape")
    ap.add_argument("--xstage-probe", action="store_true",
                    help="run the burst/gap store microbenchmark on local HBM, print the rows and the calibration, exit")
    ap.add_argument("--trace", action="store_true",
                    help="add the grouped GEMMs' per-CTA wait counters (one extra traced step) to the JSON line")
    ap.add_argument("--zero-operands", choices=["none", "weights", "all"], default="none",
                    help="power diagnostic, not a benchmark: the same launches, bytes and instructions with the expert "
                         "weights (and x) set to zero, which the 1 kW cap does not throttle")
    ap.add_argument("--profile", action="store_true",
                    help="profiler run: warm-up and timed steps only (no per-kernel pass, end-to-end or CPU legs)")
    args = ap.parse_args()

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain script: become the launcher of args.gpus ranks (one per GPU) and pass their output on
        import socket
        from paper_2607_23264_b200 import replicas
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd, extra = replicas.launcher_command(args.gpus, os.path.abspath(__file__), sys.argv[1:], port, sys.executable)
        env = dict(os.environ)
        for key, val in extra.items():
            env.setdefault(key, val)
        sys.exit(subprocess.call(cmd, env=env))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cfg = gen.CONFIGS[args.config]
    if args.tokens:
        # the same layer at another batch size (a serving batch): same seed and weights, T tokens
        import dataclasses
        cfg = dataclasses.replace(cfg, name=f"{cfg.name}@T={args.tokens}", T=args.tokens)
    if args.warmup < 3 and args.impl == "b200" and not args.sweep:
        args.warmup = 3   # timing rule: at least three warm-up steps

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_23264_b200 import binding, replicas

    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if args.probe_mma:
        pctx = binding.Context(128, 64, 64, 1, 1, device=local_rank)
        # the first launches run while the clocks ramp: warm up, then keep the smallest of several runs per point
        for _ in range(20):
            pctx.moe_probe_mma_cycles(128, 256, 16384)
        best = lambda fn: min(fn() for _ in range(7))
        rows = [{"M": M, "N": N, "clocks_per_mma": best(lambda: pctx.moe_probe_mma_cycles(M, N))}
                for M in (128, 64) for N in (16, 32, 64, 128, 256)]
        kinds = ((1, "kind::f8f6f4 (E4M3), 128xNx32"), (2, "kind::mxf8f6f4.block_scale (E4M3, E8M0 scales), 128xNx32"),
                 (3, "kind::mxf8f6f4.block_scale with 3 tcgen05.cp scale copies per 4 instructions, 128xNx32"))
        rows8 = [{"kind": name, "N": N, "clocks_per_mma": best(lambda: pctx.moe_probe_mma_cycles_kind(kind, 128, N))}
                 for kind, name in kinds for N in (32, 64, 96, 128, 192, 256)]
        print(json.dumps({"probe": "tcgen05.mma kind::f16 MxNx16, one CTA, operands resident in shared memory",
                          "rows": rows, "fp8_rows": rows8}), flush=True)
        return
    if args.xstage_probe:
        run_xstage_probe(dev)
        return
    if args.router:
        run_router(args, cfg, binding, local_rank, dev)
        return
    if args.library_gemms:
        run_library_gemms(args, cfg, dev, local_rank)
        return
    # started by a launcher (WORLD_SIZE set): join the group even as the only rank, so N = 1 takes the N-rank path
    replicas.init_process_group(world, "nccl", torch.device(dev), force="WORLD_SIZE" in os.environ)

    # every rank gets its own batch (the seeded batch, rows rotated by rank); expert weights are replicated
    x_bits = replicas.rank_batch(gen.make_x(cfg), rank)
    logits = gen.make_logits(cfg, x_bits)

    to_dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
    w_gate = torch.empty((cfg.E, cfg.F, cfg.H), dtype=torch.bfloat16, device=dev)
    w_up = torch.empty((cfg.E, cfg.F, cfg.H), dtype=torch.bfloat16, device=dev)
    w_down = torch.empty((cfg.E, cfg.H, cfg.F), dtype=torch.bfloat16, device=dev)
    want_cpu = rank == 0 and world == 1 and not (args.no_cpu_baseline or args.sweep or args.profile or args.fp8 or args.mxfp8)
    keep_host = want_cpu and cfg.E <= 16
    host_w = {}

    def sink(e, g, u, d):
        w_gate[e].copy_(to_dev(g))
        w_up[e].copy_(to_dev(u))
        w_down[e].copy_(to_dev(d))
        if keep_host:
            host_w[e] = (g, u, d)

    gen.for_each_expert(cfg, sink)
    x = to_dev(x_bits)
    if args.zero_operands != "none":
        want_cpu = False
        for w in (w_gate, w_up, w_down):
            w.zero_()
        if args.zero_operands == "all":
            x.zero_()     # the logits stay the seeded ones: same routing, same tiles
    d_logits = torch.from_numpy(logits).to(dev)
    ctx = binding.Context(cfg.T, cfg.H, cfg.F, cfg.E, cfg.k, device=local_rank)
    ws = torch.empty(ctx.workspace_bytes(), dtype=torch.uint8, device=dev)
    out = torch.empty((cfg.T, cfg.H), dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        replicas.barrier(world)
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1), world, dev)

    if args.sweep:
        run_sweep(args, cfg, ctx, binding, (x, d_logits, w_gate, w_up, w_down, out, ws), timed, rank)
        return
    if args.fp8:
        run_fp8(args, cfg, ctx, binding, (x, d_logits, w_gate, w_up, w_down, out), timed, rank, world, dev)
        return
    if args.mxfp8:
        run_mxfp8(args, cfg, ctx, binding, (x, d_logits, w_gate, w_up, w_down, out), timed, rank, world, dev)
        return

    dbg = (2 if args.one_launch else 0) | {"auto": 0, "on": 8, "off": 16}[args.pairs]
    tuning = binding.make_tuning(args.burst, args.mode, args.ik, schedule=args.schedule, dep_lead_D=args.lead,
                                 debug_flags=dbg)
    step = lambda: ctx.moe_fused_forward(x, d_logits, w_gate, w_up, w_down, out, ws, tuning=tuning)

    # ---- device-resident throughput.  Four regions, all on the launch stream:
    #   burst : args.steps steps back to back right after the warm-up (the GPU still in its boost state);
    #   heat  : at least two seconds of back-to-back steps, untimed, until the 1 kW power cap has settled the clocks;
    #   steady: args.steps steps back to back, bracketed by a barrier and a synchronize on both sides, one event
    #           between consecutive steps: ms_per_step = the whole region / steps (this is the line's value), and
    #           the median of the per-step times is reported beside it;
    #   the per-kernel times of the burst and of the steady region come from those very steps: the library records
    #           its events inside them and keeps the last 32 calls' events, which are read after the region.
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)

    def region(steps):
        """steps back-to-back steps between two barriers.  The library records its per-kernel events inside the same
        steps (a ring of the last 32 calls' events, read after the region: no host synchronisation in between), so the
        kernel times are those of the timed steps themselves and sum to no more than the step."""
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ctx.moe_set_kernel_timing(events_inside)
        barrier()
        marks[0].record(stream)
        for i in range(steps):
            step()
            marks[i + 1].record(stream)
        barrier()
        total = replicas.max_over_ranks(marks[0].elapsed_time(marks[-1]), world, dev)
        if events_inside:
            per = [ctx.moe_get_kernel_times_back(b) for b in range(min(steps, binding.TIMING_SLOTS))]
            ctx.moe_set_kernel_timing(False)
        else:       # launch-bound layer: a pass of its own, the events read after every step
            ctx.moe_set_kernel_timing(True)
            per = []
            for _ in range(steps):
                step()
                per.append(ctx.moe_get_kernel_times())
            ctx.moe_set_kernel_timing(False)
        kernels = [float(np.mean([s[i] for s in per])) for i in range(len(binding.KERNEL_NAMES))]
        return total, [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)], kernels

    # Eight event records per step cost a launch-bound layer a third of its step (65 against 44 us on the tiny
    # layer), so for steps under half a millisecond the per-kernel times come from a separate pass instead.
    probe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    probe[0].record(stream)
    for _ in range(3):
        step()
    probe[1].record(stream)
    torch.cuda.synchronize()
    events_inside = probe[0].elapsed_time(probe[1]) / 3 >= 0.5

    burst_total_ms, _, burst_kernel_ms = region(args.steps)
    launches = ctx.moe_last_launch_count() * args.steps
    if args.profile:
        if rank == 0:
            print(json.dumps({"profile_run": True, "ms_per_step": burst_total_ms / args.steps,
                              "config": workload_config(cfg, world)}), flush=True)
        if dist.is_initialized():
            dist.destroy_process_group()
        return
    if rank == 0:
        sampler.start()
    heat_t0, heat_steps = time.time(), 0
    while time.time() - heat_t0 < args.heat_seconds:
        for _ in range(10):
            step()
        heat_steps += 10
        torch.cuda.synchronize()
    total_ms, step_times, kernel_ms = region(args.steps)
    # SM clock of the steady region from the kernel itself: the Linear-1 producer's clock64 span over the kernel's
    # CUDA-event time, in one traced step taken while the GPU is still in that state (read, never set)
    ctx.moe_set_kernel_timing(True)
    ctx.moe_fused_forward(x, d_logits, w_gate, w_up, w_down, out, ws,
                          tuning=binding.make_tuning(args.burst, args.mode, args.ik, schedule=args.schedule,
                                                     dep_lead_D=args.lead, debug_flags=dbg | 1))
    span = float(ctx.moe_get_ffn_trace()[0, :, 0].max())
    ms4 = ctx.moe_get_kernel_times()[4]
    ctx.moe_set_kernel_timing(False)
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None and ms4 > 0:
        clocks["sm_mhz_kernel"] = span / (ms4 * 1e-3) / 1e6

    # per-step statistics with one event pair per step (the paper reports medians of 20 trials, Sec. 5.1); small
    # layers whose working set fits L2 are also timed cold, a 512 MB memset between steps evicting L2
    def per_step(flush):
        scrub = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if flush else None
        times = []
        for _ in range(args.steps):
            if flush:
                scrub.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            step()
            b.record(stream)
            b.synchronize()
            times.append(a.elapsed_time(b))
        return {"median_ms": statistics.median(times), "min_ms": min(times), "max_ms": max(times)}

    step_stats = {"steady": {"median_ms": statistics.median(step_times), "min_ms": min(step_times),
                             "max_ms": max(step_times), "heat_steps_before": heat_steps},
                  "synchronised_each_step": per_step(False)}
    weights_bytes = 6 * cfg.E * cfg.H * cfg.F
    if weights_bytes < (256 << 20) or cfg.T <= 256:
        step_stats["cold_l2_flushed"] = per_step(True)

    # the same step replayed from a CUDA graph (launch overhead off the critical path; matters for small layers)
    try:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            g.capture_begin()
            ctx.moe_fused_forward(x, d_logits, w_gate, w_up, w_down, out, ws, tuning=tuning, stream=side)
            g.capture_end()
        torch.cuda.synchronize()
        for _ in range(3):
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.steps):
            g.replay()
        b.record(stream)
        b.synchronize()
        step_stats["graph_replay_ms_per_step"] = a.elapsed_time(b) / args.steps
    except Exception as exc:      # a capture failure must not lose the bench line
        step_stats["graph_replay_ms_per_step"] = None
        step_stats["graph_error"] = str(exc)[:200]

    ffn_trace = None
    if args.trace:
        ttn = binding.make_tuning(args.burst, args.mode, args.ik, schedule=args.schedule, dep_lead_D=args.lead,
                                  debug_flags=dbg | 1)
        ctx.moe_fused_forward(x, d_logits, w_gate, w_up, w_down, out, ws, tuning=ttn)
        tr = ctx.moe_get_ffn_trace().astype(np.float64)          # [2, CTAs, 8]
        ffn_trace = {}
        for i, name in enumerate(("linear1", "linear2")):
            mean = tr[i].mean(axis=0)
            tiles = max(mean[6], 1.0)
            ffn_trace[name] = {f: float(v) for f, v in zip(binding.TRACE_FIELDS, mean)}
            ffn_trace[name]["per_tile_clocks"] = {f: float(v / tiles) for f, v in zip(binding.TRACE_FIELDS, mean)
                                                  if f != "tiles"}
            ffn_trace[name]["tiles_min_max"] = [float(tr[i][:, 6].min()), float(tr[i][:, 6].max())]

    code, detail = ctx.moe_last_device_status()
    if code != 0:
        raise RuntimeError(f"device status {binding.STATUS_NAMES.get(code, code)} detail {detail:#x}")

    # ---- end to end through the host-buffer entry point: H2D of x and logits, D2H of out, every step
    x_host = torch.from_numpy(x_bits.view(np.int16)).pin_memory()
    logits_host = torch.from_numpy(logits).pin_memory()
    out_host = torch.empty((cfg.T, cfg.H), dtype=torch.int16).pin_memory()
    e2e_step = lambda: ctx.moe_fused_forward_host(x_host, logits_host, w_gate, w_up, w_down, out_host, ws,
                                                  tuning=tuning)
    e2e_serial_ms = timed(e2e_step, args.steps, args.warmup)

    # the same through the two-deep pipelined entry point (copies of neighbouring steps overlap the layer);
    # the flush, inside the timed region, makes the stream wait for the last copies
    pipe_step = lambda: ctx.moe_fused_forward_host_pipelined(x_host, logits_host, w_gate, w_up, w_down, out_host, ws,
                                                             tuning=tuning)
    for _ in range(args.warmup):
        pipe_step()
    heat_t0 = time.time()                  # the same pre-heating as the device-resident region, through this entry point
    while time.time() - heat_t0 < args.heat_seconds / 2:
        for _ in range(10):
            pipe_step()
        ctx.moe_host_pipeline_flush()
        torch.cuda.synchronize()
    ctx.moe_host_pipeline_flush()
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for _ in range(args.steps):
        pipe_step()
    ctx.moe_host_pipeline_flush()
    p1.record(stream)
    barrier()
    e2e_ms = replicas.max_over_ranks(p0.elapsed_time(p1), world, dev)
    h2d = x_host.numel() * 2 + logits_host.numel() * 4
    d2h = out_host.numel() * 2

    # Context, after every timed region and on nothing the layer uses: the library bf16 GEMM of the measured-peaks file
    # (8192^3, back to back for 2 s after 1 s of the same) on the GPU at hand.  GPUs of one pool hold different clocks
    # at the same 1 kW cap; this says how the GPU of this run compares with the one the peaks were taken on.  The
    # roofline's `peak` stays the file's figure.
    local_peak, library_grouped_ms = None, None
    if rank == 0 and world == 1 and not args.no_local_peak and not args.profile:
        n = 8192
        ga = torch.randn((n, n), device=dev, dtype=torch.float32).to(torch.bfloat16)
        gb = torch.randn((n, n), device=dev, dtype=torch.float32).to(torch.bfloat16)
        gc = torch.empty((n, n), device=dev, dtype=torch.bfloat16)
        t_heat = time.time()
        while time.time() - t_heat < 1.0:
            for _ in range(20):
                torch.matmul(ga, gb, out=gc)
            torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        count, t_run = 0, time.time()
        g0.record(stream)
        while time.time() - t_run < 2.0:
            for _ in range(20):
                torch.matmul(ga, gb, out=gc)
            count += 20
            torch.cuda.synchronize()
        g1.record(stream)
        torch.cuda.synchronize()
        local_peak = 2.0 * n ** 3 * count / (g0.elapsed_time(g1) * 1e-3) / 1e12
        del ga, gb, gc
        # and the layer's own two grouped GEMMs as library calls, one per expert and weight matrix, on the very tensors
        # of the last step (x_perm, h and the expert row ranges in the workspace; no SiLU*mul): layers of few experts only
        if cfg.E <= 16:
            lay = ctx.workspace_layout()
            offs = ws[lay["offsets"]:lay["offsets"] + 4 * (cfg.E + 1)].view(torch.int32).cpu().numpy().astype(np.int64)
            xp = ws[lay["x_perm"]:lay["x_perm"] + cfg.R * cfg.H * 2].view(torch.bfloat16).view(cfg.R, cfg.H)
            hp = ws[lay["h"]:lay["h"] + cfg.R * cfg.F * 2].view(torch.bfloat16).view(cfg.R, cfg.F)
            lg = torch.empty((cfg.R, cfg.F), dtype=torch.bfloat16, device=dev)
            lu = torch.empty((cfg.R, cfg.F), dtype=torch.bfloat16, device=dev)
            ly = torch.empty((cfg.R, cfg.H), dtype=torch.bfloat16, device=dev)
            spans = [(e, int(offs[e]), int(offs[e + 1])) for e in range(cfg.E) if offs[e + 1] > offs[e]]

            def library_gemms():
                for e, lo, hi in spans:
                    torch.matmul(xp[lo:hi], w_gate[e].t(), out=lg[lo:hi])
                    torch.matmul(xp[lo:hi], w_up[e].t(), out=lu[lo:hi])
                for e, lo, hi in spans:
                    torch.matmul(hp[lo:hi], w_down[e].t(), out=ly[lo:hi])

            t_heat = time.time()
            while time.time() - t_heat < 1.0:
                library_gemms()
                torch.cuda.synchronize()
            count, t_run = 0, time.time()
            g0.record(stream)
            while time.time() - t_run < 1.5:
                for _ in range(5):
                    library_gemms()
                count += 5
                torch.cuda.synchronize()
            g1.record(stream)
            torch.cuda.synchronize()
            library_grouped_ms = g0.elapsed_time(g1) / count
            del lg, lu, ly

    if rank != 0:
        if dist.is_initialized():
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    ms_per_step = total_ms / args.steps
    tokens = cfg.T * world
    value = replicas.job_tokens_per_second(cfg.T, world, args.steps, total_ms)
    tflops = cfg.flops * world / (ms_per_step * 1e-3) / 1e12
    R = cfg.R
    l1_flops = 4 * R * cfg.H * cfg.F
    l2_flops = 2 * R * cfg.H * cfg.F
    # both GEMMs in one kernel (asked for, or chosen by the library for wave-sized layers): its time is in slot 4
    one_launch = args.schedule == 1 or args.one_launch or launches == 6 * args.steps
    if one_launch:
        l1_flops, l2_flops = l1_flops + l2_flops, 0
    l1_tf = l1_flops / (kernel_ms[4] * 1e-3) / 1e12
    l2_tf = 0.0 if one_launch else l2_flops / (kernel_ms[5] * 1e-3) / 1e12
    move_bytes = 2 * cfg.H * (cfg.T + R)
    disp_gbs = move_bytes / (kernel_ms[3] * 1e-3) / 1e9
    comb_gbs = (move_bytes + 8 * R) / (kernel_ms[6] * 1e-3) / 1e9
    peak_tf_burst = float(peaks["bf16_tflops"])
    peak_tf = float(peaks.get("bf16_tflops_sustained", peak_tf_burst))   # the steady region is a long step loop
    peak_hbm = float(peaks["hbm_gbs"])
    lay = ctx.workspace_layout()
    counts = ws[lay["counts"]:lay["counts"] + 4 * cfg.E].view(torch.int32).cpu().numpy()
    nonempty = int((counts > 0).sum())
    # algorithmic bytes of one Linear-1 launch: gate+up weights of the non-empty experts, x_perm read, h written
    l1_bytes = nonempty * 2 * cfg.F * cfg.H * 2 + R * cfg.H * 2 + R * cfg.F * 2
    l2_bytes = nonempty * cfg.F * cfg.H * 2 + R * cfg.F * 2 + R * cfg.H * 2
    if one_launch:
        l1_bytes, l2_bytes = l1_bytes + l2_bytes, 0
    l1_gbs = l1_bytes / (kernel_ms[4] * 1e-3) / 1e9
    l2_gbs = 0.0 if one_launch else l2_bytes / (kernel_ms[5] * 1e-3) / 1e9
    pair_kernel = not one_launch and args.pairs == "on"      # "auto": the library's default, the single-CTA kernel
    kernel_symbol = "expert_ffn_pair_kernel<false>" if pair_kernel else "expert_ffn_kernel<false>"
    gemm_name = (kernel_symbol + " (Linear-1 + SiLU*mul + Linear-2, one launch)" if one_launch
                 else kernel_symbol + ", Linear-1 + SiLU*mul launch")
    per_expert = None if one_launch else dram_traffic_per_expert(kernel_symbol, cfg.H, cfg.F)
    traffic = None if per_expert is None else per_expert * nonempty
    # the roofline that binds Linear-1: tensor time at the measured GEMM peak vs HBM time at the measured copy rate
    t_tensor = l1_flops / (peak_tf_burst * 1e12)
    t_hbm = l1_bytes / (peak_hbm * 1e9)
    burst_ms4 = burst_kernel_ms[4]
    if t_tensor >= t_hbm:
        burst_tf = l1_flops / (burst_ms4 * 1e-3) / 1e12
        roofline = {
            "kernel": gemm_name, "bound": "tensor", "achieved": l1_tf,
            "peak": peak_tf, "unit": "TFLOP/s", "frac": l1_tf / peak_tf, "traffic": traffic,
            "peak_source": f"{peak_kind} bf16_tflops_sustained (cuBLAS in a seconds-long loop): the kernel is timed inside "
                           "a pre-heated loop of steps",
            "flops_per_launch": l1_flops, "ms_per_launch": kernel_ms[4],
            "burst": {"achieved": burst_tf, "peak": peak_tf_burst, "frac": burst_tf / peak_tf_burst,
                      "ms_per_launch": burst_ms4, "peak_source": f"{peak_kind} bf16_tflops (burst)"},
        }
    else:
        roofline = {
            "kernel": gemm_name, "bound": "hbm", "achieved": l1_gbs,
            "peak": peak_hbm, "unit": "GB/s", "frac": l1_gbs / peak_hbm, "traffic": traffic,
            "peak_source": f"{peak_kind} hbm_gbs (copy)",
            "bytes_per_launch": l1_bytes, "ms_per_launch": kernel_ms[4], "nonempty_experts": nonempty,
            "tensor_tflops": l1_tf,
            "burst": {"achieved": l1_bytes / (burst_ms4 * 1e-3) / 1e9, "peak": peak_hbm,
                      "frac": l1_bytes / (burst_ms4 * 1e-3) / 1e9 / peak_hbm, "ms_per_launch": burst_ms4},
        }
    if traffic is not None:
        roofline["traffic_source"] = ("profiles/linear1_dram_traffic.md: ncu dram read + write bytes per non-empty expert "
                                      f"of {kernel_symbol} on its profiler-sized case x {nonempty} experts")
    # The cuBLAS peak was measured at its own SM clock under the power cap; this kernel ran at sm_mhz_kernel (its
    # clock64 span over its CUDA-event time).  frac x (peak's clock / this clock) compares flops per clock.
    peak_mhz = float((peaks.get("clocks_under_load") or {}).get("sm_mhz_median") or 0.0)
    if roofline["bound"] == "tensor" and peak_mhz > 0 and clocks and clocks.get("sm_mhz_kernel"):
        roofline["peak_sm_mhz"] = peak_mhz
        roofline["frac_at_equal_clock"] = roofline["frac"] * peak_mhz / clocks["sm_mhz_kernel"]
    if local_peak is not None:
        roofline["local_library_gemm"] = {
            "bf16_tflops_sustained_this_gpu": local_peak,
            "how": "torch.matmul bf16 8192^3 back to back for 2 s after 1 s of the same, after all timed regions",
            "of_measured_peaks_file": local_peak / float(peaks.get("bf16_tflops_sustained") or float("nan")),
            **({"frac_of_this_gpu": roofline["achieved"] / local_peak} if roofline["bound"] == "tensor" else {}),
            **({"grouped_gemms_as_library_calls_ms": library_grouped_ms,
                "grouped_gemms_this_build_ms": kernel_ms[4] + kernel_ms[5],
                "grouped_how": "torch.matmul per expert and weight matrix on the step's own x_perm, h and expert row "
                               "ranges (no SiLU*mul), back to back for 1.5 s after 1 s of the same; this build's figure "
                               "is its two GEMM kernels in the steady region"}
               if library_grouped_ms is not None else {})}
    burst_ms_per_step = burst_total_ms / args.steps
    line = {
        "metric": "fused MoE fwd tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic" if args.zero_operands == "none" else
                f"synthetic routing, ZERO {args.zero_operands} operands: power diagnostic, not a benchmark figure",
        "config": workload_config(cfg, world),
        "tflops": tflops, "frac_bf16_peak": tflops / world / peak_tf, "frac_bf16_peak_of": "bf16_tflops_sustained",
        "burst_ms_per_step": burst_ms_per_step, "burst_value": cfg.T * world / (burst_ms_per_step * 1e-3),
        "burst_frac_bf16_peak": cfg.flops / (burst_ms_per_step * 1e-3) / 1e12 / peak_tf_burst,
        "timed_region": f"{args.steps} back-to-back steps after {heat_steps} untimed pre-heating steps "
                        f"({args.heat_seconds:.1f} s); burst_* = {args.steps} steps right after the warm-up",
        "kernels_ms": dict(zip(binding.KERNEL_NAMES, kernel_ms)),
        "kernels_ms_source": ("the timed steady steps themselves (library events inside the region)" if events_inside
                              else "a separate pass after the region (launch-bound layer)"),
        "burst_kernels_ms": dict(zip(binding.KERNEL_NAMES, burst_kernel_ms)),
        "linear2_tflops": l2_tf, "linear1_gbs": l1_gbs, "linear2_gbs": l2_gbs, "dispatch_gbs": disp_gbs, "combine_gbs": comb_gbs,
        "dispatch_frac_hbm": disp_gbs / float(peaks["hbm_gbs"]), "combine_frac_hbm": comb_gbs / float(peaks["hbm_gbs"]),
        "roofline": roofline,
        "e2e": {"value": tokens / (e2e_ms / args.steps * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps,
                "api": "moe_fused_forward_host_pipelined + moe_host_pipeline_flush (two staging slots), timed after "
                       "pre-heating through the same entry point",
                "serial_ms_per_step": e2e_serial_ms / args.steps,
                "serial_value": tokens / (e2e_serial_ms / args.steps * 1e-3)},
        "per_step": step_stats, "gpu_launches": launches, "clocks": clocks, "tuning": [args.burst, args.mode, args.ik],
        "schedule": {"schedule": args.schedule, "lead_D": args.lead, "one_launch": one_launch},
    }
    if ffn_trace is not None:
        line["ffn_trace"] = ffn_trace
    if keep_host:
        rate, dt = oracle_sample_rate(cfg, x_bits, logits, lambda e: host_w[e], args.cpu_baseline_tokens)
        line["cpu_baseline"] = {
            "value": rate, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{min(args.cpu_baseline_tokens, cfg.T)} seeded-random tokens of {cfg.name} (row-sampled fp64 "
                      f"oracle, {dt:.1f} s; the oracle's widening of each touched expert's bf16 matrices to fp64 is part "
                      "of the timed call)"}
    elif want_cpu:
        # many experts: sample tokens until they touch about 64 experts, regenerate those experts' weights on the
        # host first (input generation, not timed), then time the oracle on the sample
        from oracle import moe_oracle as orc
        ids, _ = orc.topk_route(logits, cfg.k)
        rng = np.random.default_rng(1234)
        toks, experts = [], set()
        for t in rng.permutation(cfg.T):
            toks.append(int(t))
            experts.update(ids[t].tolist())
            if len(experts) >= 64 or len(toks) >= args.cpu_baseline_tokens:
                break
        stream_w = gen.WeightStream(cfg, sorted(experts))
        held = {e: stream_w(e) for e in sorted(experts)}
        stream_w.close()
        toks = np.sort(np.array(toks))
        t0 = time.perf_counter()
        orc.forward_tokens(toks, x_bits, logits, cfg.k, lambda e: held[e])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": len(toks) / dt, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{len(toks)} seeded-random tokens of {cfg.name} touching {len(experts)} experts "
                      f"(row-sampled fp64 oracle, {dt:.1f} s)"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if dist.is_initialized():
        dist.destroy_process_group()


def preheat(step, seconds):
    """Back-to-back untimed steps for `seconds`, until the power cap has settled the clocks."""
    import torch
    t0 = time.time()
    while time.time() - t0 < seconds:
        for _ in range(10):
            step()
        torch.cuda.synchronize()


def run_fp8(args, cfg, ctx, binding, bufs, timed, rank, world, dev):
    """The FP8 (E4M3, W8A8) variant: same layer, same algorithmic flops, experts in E4M3 with row scales."""
    import torch
    x, d_logits, w_gate, w_up, w_down, out = bufs
    wq = []
    for w in (w_gate, w_up, w_down):
        E, r, c = w.shape
        codes = torch.empty((E * r, c), dtype=torch.uint8, device=dev)
        scales = torch.empty((E * r,), dtype=torch.float32, device=dev)
        ctx.moe_quantize_rows(w.view(E * r, c), E * r, c, codes, scales)
        wq += [codes, scales]
    torch.cuda.synchronize()
    del w_gate, w_up, w_down
    ws = torch.empty(ctx.workspace_layout_fp8()["total"], dtype=torch.uint8, device=dev)
    tn = binding.make_tuning(args.burst, args.mode, args.ik, debug_flags={"auto": 0, "on": 8, "off": 16}[args.pairs])
    step = lambda: ctx.moe_fused_forward_fp8(x, d_logits, *wq, out, ws, tuning=tn)
    sampler = ClockSampler(torch.cuda.current_device())
    burst_ms = timed(step, args.steps, args.warmup) / args.steps
    if rank == 0:
        sampler.start()
    preheat(step, args.heat_seconds)
    ms = timed(step, args.steps, 0) / args.steps
    ctx.moe_set_kernel_timing(True)
    per = []
    for _ in range(args.steps):
        step()
        per.append(ctx.moe_get_kernel_times())
    ctx.moe_set_kernel_timing(False)
    clocks = sampler.stop() if rank == 0 else None
    km = [float(np.mean([p[i] for p in per])) for i in range(len(binding.KERNEL_NAMES))]
    waits = None
    if args.trace:
        # one traced step: the GEMMs' own wait counters, averaged over CTAs, as shares of the producer's span
        ttn = binding.make_tuning(args.burst, args.mode, args.ik,
                                  debug_flags={"auto": 0, "on": 8, "off": 16}[args.pairs] | 1)
        ctx.moe_fused_forward_fp8(x, d_logits, *wq, out, ws, tuning=ttn)
        tr = ctx.moe_get_ffn_trace().astype(np.float64)
        waits = {}
        for gi, gname in enumerate(("linear1", "linear2")):
            live = tr[gi, :, 0] > 0
            span = np.maximum(tr[gi, live, 0], 1.0)
            waits[gname] = {"span_clocks": float(span.mean()), "tiles_per_cta": float(tr[gi, live, 6].mean()),
                            "mma_waits_operands": float((tr[gi, live, 2] / span).mean()),
                            "mma_waits_accumulator": float((tr[gi, live, 3] / span).mean()),
                            "producer_waits_stage": float((tr[gi, live, 1] / span).mean()),
                            "epilogue_busy": float((tr[gi, live, 5] / span).mean())}
    code, detail = ctx.moe_last_device_status()
    if code != 0:
        raise RuntimeError(f"device status {code} detail {detail:#x}")
    if rank != 0:
        return
    peaks, kind = load_peaks()
    peak = 2.0 * float(peaks["bf16_tflops"])      # E4M3 runs at twice the bf16 rate on this part (4.5 vs 2.25 PFLOP/s nominal)
    R = cfg.R
    l1_tf = 4 * R * cfg.H * cfg.F / (km[4] * 1e-3) / 1e12
    tflops = cfg.flops * world / (ms * 1e-3) / 1e12
    line = {
        "metric": "fused MoE fwd tokens/s", "variant": "fp8 (E4M3 W8A8, per-row scales)", "value": cfg.T * world / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "burst_ms_per_step": burst_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3", "data": "synthetic",
        "config": workload_config(cfg, world), "tflops": tflops, "frac_fp8_peak": tflops / world / peak,
        "kernels_ms": {"routing": km[0] + km[1] + km[2], "quantize_x+dispatch": km[3], "linear1": km[4],
                       "quantize_h+linear2": km[5], "combine": km[6]},
        "roofline": {"kernel": "expert FFN Linear-1 launch, E4M3 operands", "bound": "tensor", "achieved": l1_tf,
                     "peak": peak, "unit": "TFLOP/s", "frac": l1_tf / peak, "traffic": None,
                     "peak_source": f"2 x {kind} bf16_tflops (burst): nominal fp8 / bf16 ratio"},
        "gpu_launches": ctx.moe_last_launch_count() * args.steps, "clocks": clocks, "gemm_waits": waits,
    }
    print(json.dumps(line), flush=True)


def run_mxfp8(args, cfg, ctx, binding, bufs, timed, rank, world, dev):
    """The block-scaled FP8 variant (MXFP8: E4M3 elements, E8M0 scale per 32 elements along K, applied inside the MMA)."""
    import torch
    x, d_logits, w_gate, w_up, w_down, out = bufs
    wq = []
    for w in (w_gate, w_up, w_down):
        E, r, c = w.shape
        codes = torch.empty((E * r, c), dtype=torch.uint8, device=dev)
        words = torch.empty((c // 128, E * r), dtype=torch.int32, device=dev)
        ctx.moe_quantize_rows_mx(w.view(E * r, c), E * r, c, codes, words)
        wq += [codes, words]
    torch.cuda.synchronize()
    del w_gate, w_up, w_down
    ws = torch.empty(ctx.workspace_layout_mx()["total"], dtype=torch.uint8, device=dev)
    step = lambda: ctx.moe_fused_forward_mx(x, d_logits, *wq, out, ws)
    sampler = ClockSampler(torch.cuda.current_device())
    burst_ms = timed(step, args.steps, args.warmup) / args.steps
    if rank == 0:
        sampler.start()
    preheat(step, args.heat_seconds)
    ms = timed(step, args.steps, 0) / args.steps
    ctx.moe_set_kernel_timing(True)
    per = []
    for _ in range(args.steps):
        step()
        per.append(ctx.moe_get_kernel_times())
    ctx.moe_set_kernel_timing(False)
    clocks = sampler.stop() if rank == 0 else None
    km = [float(np.mean([p[i] for p in per])) for i in range(len(binding.KERNEL_NAMES))]
    # the GEMMs' own wait counters (recorded while per-kernel timing is on), averaged over CTAs, as shares of the span
    tr = ctx.moe_get_ffn_trace().astype(np.float64)
    waits = {}
    for gi, gname in enumerate(("linear1", "linear2")):
        span = np.maximum(tr[gi, :, 0], 1.0)
        waits[gname] = {"span_clocks": float(span.mean()), "tiles_per_cta": float(tr[gi, :, 6].mean()),
                        "mma_waits_operands": float((tr[gi, :, 2] / span).mean()),
                        "mma_waits_accumulator": float((tr[gi, :, 3] / span).mean()),
                        "producer_waits_stage": float((tr[gi, :, 1] / span).mean()),
                        "epilogue_busy": float((tr[gi, :, 5] / span).mean()),
                        "swapped_tiles_per_cta": float(tr[gi, :, 8].mean()),
                        "clocks_per_swapped_tile": float(tr[gi, :, 9].sum() / max(tr[gi, :, 8].sum(), 1.0)),
                        "clocks_per_other_tile": float(tr[gi, :, 11].sum() / max((tr[gi, :, 6] - tr[gi, :, 8]).sum(), 1.0))}
    code, detail = ctx.moe_last_device_status()
    if code != 0:
        raise RuntimeError(f"device status {code} detail {detail:#x}")
    if rank != 0:
        return
    peaks, kind = load_peaks()
    peak = 2.0 * float(peaks["bf16_tflops"])      # E4M3 runs at twice the bf16 rate on this part (4.5 vs 2.25 PFLOP/s nominal)
    R = cfg.R
    l1_tf = 4 * R * cfg.H * cfg.F / (km[4] * 1e-3) / 1e12
    tflops = cfg.flops * world / (ms * 1e-3) / 1e12
    line = {
        "metric": "fused MoE fwd tokens/s", "variant": "mxfp8 (E4M3 elements, E8M0 scale per 32 along K)",
        "value": cfg.T * world / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "burst_ms_per_step": burst_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "mxfp8_e4m3", "data": "synthetic",
        "config": workload_config(cfg, world), "tflops": tflops, "frac_fp8_peak": tflops / world / peak,
        "kernels_ms": {"routing": km[0] + km[1] + km[2], "quantize_x+dispatch": km[3], "linear1+quantize_h": km[4],
                       "linear2": km[5], "combine": km[6]},
        "roofline": {"kernel": "expert FFN Linear-1 launch, block-scaled E4M3 operands", "bound": "tensor",
                     "achieved": l1_tf, "peak": peak, "unit": "TFLOP/s", "frac": l1_tf / peak, "traffic": None,
                     "peak_source": f"2 x {kind} bf16_tflops (burst): nominal fp8 / bf16 ratio"},
        "gpu_launches": ctx.moe_last_launch_count() * args.steps, "clocks": clocks, "gemm_waits": waits,
    }
    print(json.dumps(line), flush=True)


def run_library_gemms(args, cfg, dev, local_rank):
    """What the two grouped GEMMs cost as library calls on this GPU: one torch.matmul per non-empty expert and weight
    matrix over that expert's rows of the seeded routing.  Random operands of the layer's distributions (timing does
    not depend on the values beyond their statistics); no SiLU*mul, routing, dispatch or combine.  Context for the
    bench line of the same workload: both sit under the same 1 kW cap on the same GPU."""
    import torch
    from paper_2607_23264_b200 import binding
    R, H, F = cfg.R, cfg.H, cfg.F
    x_bits = gen.make_x(cfg)
    d_logits = torch.from_numpy(gen.make_logits(cfg, x_bits)).to(dev)
    ctx = binding.Context(cfg.T, H, F, cfg.E, cfg.k, device=local_rank)      # the library's own routing plan: row ranges
    i32 = lambda n: torch.empty(n, dtype=torch.int32, device=dev)
    d_counts, d_offs = i32(cfg.E), i32(cfg.E + 1)
    ctx.moe_plan_routing(d_logits, i32(R), torch.empty(R, dtype=torch.float32, device=dev), d_counts, d_offs, i32(R), i32(R))
    torch.cuda.synchronize()
    counts, offs = d_counts.cpu().numpy(), d_offs.cpu().numpy().astype(np.int64)
    gsd = torch.Generator(device=dev).manual_seed(cfg.seed)
    rnd = lambda shape, std: (torch.randn(shape, generator=gsd, device=dev, dtype=torch.float32) * std).to(torch.bfloat16)
    live = [e for e in range(cfg.E) if counts[e] > 0]
    xp, hp = rnd((R, H), 1.0), rnd((R, F), 0.5)
    wg = {e: rnd((F, H), H ** -0.5) for e in live}
    wu = {e: rnd((F, H), H ** -0.5) for e in live}
    wd = {e: rnd((H, F), F ** -0.5) for e in live}
    g, u = torch.empty((R, F), dtype=torch.bfloat16, device=dev), torch.empty((R, F), dtype=torch.bfloat16, device=dev)
    y = torch.empty((R, H), dtype=torch.bfloat16, device=dev)

    def linear1():
        for e in live:
            lo, hi = int(offs[e]), int(offs[e + 1])
            torch.matmul(xp[lo:hi], wg[e].t(), out=g[lo:hi])
            torch.matmul(xp[lo:hi], wu[e].t(), out=u[lo:hi])

    def linear2():
        for e in live:
            lo, hi = int(offs[e]), int(offs[e + 1])
            torch.matmul(hp[lo:hi], wd[e].t(), out=y[lo:hi])

    def sustained(fn):
        t0 = time.time()
        while time.time() - t0 < max(args.heat_seconds, 1.0):
            fn()
            torch.cuda.synchronize()
        sampler = ClockSampler(local_rank)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n, t0 = 0, time.time()
        e0.record()
        while time.time() - t0 < 2.0:
            for _ in range(5):
                fn()
            n += 5
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n, sampler.stop()

    ms1, _ = sustained(linear1)
    ms2, _ = sustained(linear2)
    ms12, clocks = sustained(lambda: (linear1(), linear2()))
    print(json.dumps({
        "library_gemms": "torch.matmul bf16, one call per non-empty expert and weight matrix, rows of the seeded routing",
        "config": workload_config(cfg, 1), "nonempty_experts": len(live),
        "linear1_ms": ms1, "linear2_ms": ms2, "both_ms": ms12,
        "linear1_tflops": 4.0 * R * H * F / (ms1 * 1e-3) / 1e12, "linear2_tflops": 2.0 * R * H * F / (ms2 * 1e-3) / 1e12,
        "both_tflops": 6.0 * R * H * F / (ms12 * 1e-3) / 1e12, "clocks": clocks,
        "note": "GEMMs only (no SiLU*mul, routing, dispatch, combine); context for the bench line, not a product path"}),
        flush=True)


def run_router(args, cfg, binding, local_rank, dev):
    """Router front end alone: x and the prepared router weights resident on the device."""
    import torch
    x_bits = gen.make_x(cfg)
    w_router = gen.make_router(cfg)
    bias = gen.zipf_log_bias(cfg.E).astype(np.float32) if cfg.router == "xWr_zipf" else None
    ctx = binding.Context(cfg.T, cfg.H, cfg.F, cfg.E, cfg.k, device=local_rank)
    x = torch.from_numpy(np.ascontiguousarray(x_bits).view(np.int16)).to(dev).view(torch.bfloat16)
    d_w = torch.from_numpy(w_router).to(dev)
    d_bias = torch.from_numpy(bias).to(dev) if bias is not None else None
    w_split = torch.zeros(ctx.router_weight_bytes() // 2, dtype=torch.bfloat16, device=dev)
    scratch = torch.empty(ctx.router_scratch_bytes() // 4, device=dev)
    ctx.moe_router_prepare(d_w, w_split)
    R = cfg.T * cfg.k
    i32 = dict(dtype=torch.int32, device=dev)
    ids, w = torch.empty((cfg.T, cfg.k), **i32), torch.empty((cfg.T, cfg.k), device=dev)
    counts, offsets = torch.empty(cfg.E, **i32), torch.empty(cfg.E + 1, **i32)
    perm, inv_perm = torch.empty(R, **i32), torch.empty(R, **i32)
    logits = torch.empty((cfg.T, cfg.E), device=dev)
    # several copies of x, more than L2 in total, used in turn: every timed call reads its activations from HBM while
    # the calls queue back to back (no host gap inside the timed region)
    n_rot = max(2, -(-(256 << 20) // max(1, x.numel() * 2)))
    n_rot = min(n_rot, 64)
    xs = [x] + [x.clone() for _ in range(n_rot - 1)]
    l2_note = (f"{n_rot} copies of x used in turn ({n_rot * x.numel() * 2 >> 20} MiB)" if n_rot * x.numel() * 2 >= (256 << 20)
               else f"{n_rot} copies of x used in turn; they fit in L2 (warm)")
    ctx.moe_route_tokens(x, w_split, d_bias, scratch, logits, ids, w, counts, offsets, perm, inv_perm)
    routed = lambda i, st=None: ctx.moe_route_tokens(xs[i % n_rot], w_split, d_bias, scratch, None, ids, w, counts,
                                                     offsets, perm, inv_perm, stream=st)
    plain = lambda i, st=None: ctx.moe_plan_routing(logits, ids, w, counts, offsets, perm, inv_perm, stream=st)
    rows = {}
    stream = torch.cuda.current_stream()
    for name, fn in (("route_tokens", routed), ("plan_routing_from_logits", plain)):
        for i in range(args.warmup):
            fn(i)
        torch.cuda.synchronize()
        # one CUDA graph holding n_rot calls (each on its own copy of x): replaying it keeps the host's launch cost
        # out of the timed region, which for calls this short would otherwise be most of it
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            g.capture_begin()
            for i in range(n_rot):
                fn(i, side)
            g.capture_end()
        torch.cuda.synchronize()
        for _ in range(args.warmup):
            g.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            g.replay()
        e1.record(stream)
        torch.cuda.synchronize()
        rows[name] = {"call_us": e0.elapsed_time(e1) * 1e3 / (args.steps * n_rot)}
    code, detail = ctx.moe_last_device_status()
    epad = ctx.router_weight_bytes() // (2 * cfg.H * 2)
    alg_bytes = 2 * cfg.T * cfg.H + 2 * 2 * epad * cfg.H + 8 * R
    # the calls share the plan's scan and scatter; what the front end adds is the difference
    us = rows["route_tokens"]["call_us"]
    peaks, peaks_src = load_peaks()
    print(json.dumps({
        "router": True, "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "E": cfg.E, "k": cfg.k,
                                   "l2": l2_note},
        "steps": args.steps, "warmup": args.warmup, "dtype": "bf16 x (2 bf16 terms of fp32 W_r), fp32 accumulate",
        "timings": rows, "device_status": code,
        "route_tokens_call": {"us": us, "algorithmic_bytes": alg_bytes, "GBps": alg_bytes / us * 1e-3,
                          "frac_hbm": alg_bytes / us * 1e-3 / peaks["hbm_gbs"], "peaks": peaks_src,
                          "tflops_bf16_issued": 2.0 * 2 * cfg.T * cfg.H * epad / us * 1e-6},
    }), flush=True)


def run_xstage_probe(dev):
    """Periodic-burst gap sweep, zero-gap decompositions and isolated bursts on this GPU's own HBM."""
    import torch
    from paper_2607_23264_b200 import xstage
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    buf = torch.empty(1 << 30, dtype=torch.uint8, device=dev)          # 1 GiB: slices of 7 MB per producer, far above L2
    KiB = 1024
    med = lambda xs: statistics.median(xs)
    out = {"probe": "xstage_store_probe: K producers x B bytes of 16-byte stores, gap G, local HBM", "sms": sms}
    xstage.xstage_store_probe(sms, 8 * KiB, 0, 50, buf)                # warm-up
    periodic = []
    for B in (8 * KiB, 32 * KiB, 128 * KiB):
        for gap in (0, 250, 500, 1000, 2000, 4000, 8000, 16000, 32000):
            r = xstage.xstage_store_probe(sms, B, gap, 300, buf)
            tail = slice(100, 300)
            periodic.append({"producers": sms, "bytes_per_producer": B, "volume": sms * B, "gap": gap,
                             "t_iss": med(r["issue_mean"][tail]), "t_iss_max": med(r["issue_max"][tail]),
                             "t_period": med(r["period_mean"][tail]), "clocks_per_us": r["clocks_per_us"]})
    out["periodic"] = periodic
    decomp = []
    for K, B in ((sms, 32 * KiB), (sms // 2, 64 * KiB), (sms // 4, 128 * KiB)):
        r = xstage.xstage_store_probe(K, B, 0, 300, buf)
        tp = med(r["period_mean"][100:300])
        decomp.append({"producers": K, "bytes_per_producer": B, "volume": K * B, "t_period": tp,
                       "bytes_per_clock": K * B / tp, "gb_per_s": K * B / tp * r["clocks_per_us"] / 1e3})
    out["zero_gap_decompositions"] = decomp
    isolated = []
    sizes = [b * KiB for b in (1, 2, 4, 8, 12, 16, 20, 24, 28, 32, 40, 48, 64, 96, 128, 256, 512, 1024, 2048, 4096)]
    for B in sizes:
        runs = [xstage.xstage_store_probe(sms, B, 0, 1, buf) for _ in range(9)]
        isolated.append({"producers": sms, "bytes_per_producer": B, "volume": sms * B,
                         "t_iss": med([x["issue_mean"][0] for x in runs]), "t_iss_max": med([x["issue_max"][0] for x in runs])})
    out["isolated"] = isolated
    cal = {}
    for B in (8 * KiB, 32 * KiB, 128 * KiB):
        rows = [r for r in periodic if r["bytes_per_producer"] == B]
        c = xstage.calibrate(rows, isolated)
        cpu = med([r["clocks_per_us"] for r in rows])
        c["clocks_per_us"] = cpu
        c["rate_gb_per_s"] = c["rate"] * cpu / 1e3 if c["rate"] else None
        c["t_iss0_us"] = c["t_iss0"] / cpu
        if c["rate"]:
            c["recovery_gap_clocks"] = xstage.xstage_recovery_gap(c["t_iss0"], c["rate"], sms * B)
        cal[str(B)] = c
    out["calibration_by_bytes_per_producer"] = cal
    print(json.dumps(out), flush=True)


def run_sweep(args, cfg, ctx, binding, bufs, timed, rank):
    """Store-pacing sweep: burst in {1,2,4,8,16} x {after-mainloop, every-k-iterations k in {1,2,4}}.

    The GPU is first brought to its steady power-capped state (about 1.5 s of steps); every point is then
    timed in two passes (forward and reverse order) so that clock drift shows up as spread, not as a trend.
    Per point: median/min ms per step, TFLOP/s, algorithmic HBM GB/s, per-kernel times, and from one traced step
    the share of each GEMM's span its tensor pipe did useful work (the GEMM's multiply-adds over the 4096 per clock
    and SM the pipe can do, over the launch's mean CTA span), the Linear-2 per-tile epilogue store span, pacing hold and MMA wait for a free
    accumulator (SM clocks), and how many CTAs held stores at all."""
    import torch
    x, d_logits, w_gate, w_up, w_down, out, ws = bufs
    dbg = {"auto": 0, "on": 8, "off": 16}[args.pairs]
    points = [(b, 0, 1) for b in (1, 2, 4, 8, 16)] + [(b, 1, ik) for b in (1, 2, 4, 8, 16) for ik in (1, 2, 4)]
    run = lambda tn: ctx.moe_fused_forward(x, d_logits, w_gate, w_up, w_down, out, ws, tuning=tn)
    t0 = time.time()
    while time.time() - t0 < 1.5:
        for _ in range(20):
            run(None)
        torch.cuda.synchronize()
    base = None
    samples = {pt: [] for pt in points}
    extra = {}
    R = cfg.R
    step_bytes = (6 * cfg.E * cfg.H * cfg.F + 2 * (2 * cfg.T * cfg.H + 4 * R * cfg.H + 2 * R * cfg.F))
    k_blocks = (cfg.H // 64, cfg.F // 64)
    for order in (points, points[::-1]):
        for pt in order:
            tn = binding.make_tuning(*pt, debug_flags=dbg)
            ms = timed(lambda: run(tn), args.steps, max(1, args.warmup)) / args.steps
            samples[pt].append(ms)
            if pt not in extra:
                ctx.moe_set_kernel_timing(True)
                run(tn)
                km = ctx.moe_get_kernel_times()
                ctx.moe_set_kernel_timing(False)
                bits = out.view(torch.int16).clone()
                if base is None:
                    base = bits
                run(binding.make_tuning(*pt, debug_flags=dbg | 1))
                tr = ctx.moe_get_ffn_trace().astype(np.float64)
                pipe = []
                for gi in (0, 1):
                    issuing = tr[gi][:, 6] > 0           # CTAs whose MMA warp issued (in a CTA pair: the leader)
                    span = np.maximum(tr[gi][issuing, 0], 1.0)
                    # useful multiply-adds of the GEMM over what the launch's SMs could issue in its span (an SM's tensor
                    # pipe does 128 x 256 x 16 bf16 multiply-adds in 128 clocks = 4096 per clock); padded rows not counted
                    macs = (2 if gi == 0 else 1) * cfg.R * cfg.H * cfg.F
                    pipe.append(float(macs / (tr[gi].shape[0] * 4096.0 * span.mean())) if issuing.any() else 0.0)
                l2 = tr[1].mean(axis=0)
                tiles = max(tr[1][:, 6].sum() / max((tr[1][:, 5] > 0).sum(), 1), 1.0)   # tiles per draining CTA
                extra[pt] = {"linear1_ms": km[4], "linear2_ms": km[5], "identical_bits": bool(torch.equal(bits, base)),
                             "tensor_pipe_linear1": pipe[0], "tensor_pipe_linear2": pipe[1],
                             "ctas_holding_stores": [int((tr[0][:, 7] > 0).sum()), int((tr[1][:, 7] > 0).sum())],
                             "l1_pacing_hold_clk_per_cta": float(tr[0][:, 7].mean()),
                             "l2_store_span_clk_per_tile": l2[5] / tiles, "l2_pacing_hold_clk_per_tile": l2[7] / tiles,
                             "l2_mma_wait_accumulator_clk_per_tile": l2[3] / tiles,
                             "l2_mma_wait_operands_frac": l2[2] / max(l2[0], 1.0)}
    rows = []
    for pt in points:
        ms = statistics.median(samples[pt])
        e = extra[pt]
        pipe_step = (e["tensor_pipe_linear1"] * e["linear1_ms"] + e["tensor_pipe_linear2"] * e["linear2_ms"]) / ms
        rows.append({"burst": pt[0], "mode": pt[1], "k": pt[2], "ms_per_step": ms, "ms_min": min(samples[pt]),
                     "ms_max": max(samples[pt]), "tflops": cfg.flops / (ms * 1e-3) / 1e12,
                     "hbm_gbs_algorithmic": step_bytes / (ms * 1e-3) / 1e9, "tensor_pipe_step": pipe_step, **e})
    if rank == 0:
        print(json.dumps({"sweep": rows, "config": workload_config(cfg, 1), "steps_per_sample": args.steps,
                          "pairs": args.pairs}), flush=True)


if __name__ == "__main__":
    main()
