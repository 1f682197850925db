#!/usr/bin/env python
"""Benchmark of the MXFP8 hot path on B200: one training step of a linear layer.

One pass of the whole path over one batch of synthetic input, for the ~800M-parameter GPT-style
linear layer (tokens 8192, hidden 2048, FFN 8192): the three BF16 tensors X, W, dY are each
converted to MXFP8-E4M3 in both block orientations (one read each), then FPROP, DGRAD and WGRAD run
as block-scaled MXFP8 GEMMs with BF16 output.  A pass takes 0.4 ms, far too short to time alone, so
a "step" is PASSES_PER_STEP = 64 such passes back to back (64 micro-batches): the default 20 steps
then keep the device busy for half a second, which is the power-capped steady state; the first 20
passes after an idle gap are reported beside it as the burst figure.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line on rank 0.  `value` is the step's GEMM work (3 x 2MNK FLOP) divided by
the whole step time (casts included), summed over ranks; `cast` and `gemm` give the two parts
of the metric separately (GB/s and TFLOP/s from per-launch CUDA events); `roofline` describes
the dominant kernel (the GEMM); `cpu_baseline` is the CPU oracle timed on a bounded sample.
With --impl reference the oracle alone is timed (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

T, H, F = 8192, 2048, 8192          # tokens, hidden, FFN of the benchmarked linear layer
METRIC = "MXFP8 cast GB/s (% HBM peak); MXFP8 GEMM TFLOP/s (% dense FP8 peak)"
WORKLOAD = "linear layer of a ~800M-param GPT: tokens 8192, hidden 2048, FFN 8192; quantize X,W,dY (both orientations) + fprop/dgrad/wgrad MXFP8 GEMMs, BF16 out"
L2_NOTE = "inputs larger than L2: 192 MB of BF16 sources and 590 MB of outputs per pass"
NOMINAL_FP8_TFLOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/: the FPROP GEMM of this step, and the quantize kernel on a
# 128 MB BF16 tensor (the size of dY, the largest cast of the step).  Writes still dirty in
# L2 when the kernel ends are not counted by ncu, so both are below the algorithmic bytes.
NCU_TRAFFIC_GEMM_FPROP = 50.0e6 + 86.2e6
NCU_TRAFFIC_GEMM_MULTI = 333.1e6 + 153.4e6          # the three-product launch of the step (dram read + write, ncu)
NCU_TRAFFIC_QUANTIZE_STEP = 201.4e6 + 152.6e6       # the batched cast of X, W, dY (408.9 MB algorithmic; part of the output still in L2)

PASSES_PER_STEP = 64                                  # micro-batches per timed step (see the module docstring)
STEP_FLOP = 3 * 2.0 * T * H * F                       # one pass: three GEMMs of 275 GFLOP
CAST_BYTES = (T * H + F * H + T * F) * (2 + 2 * (1 + 1 / 32))   # src + two orientations x (q + scales)
GEMM_SHAPES = {"fprop": (T, F, H), "dgrad": (T, H, F), "wgrad": (F, H, T)}


def bench_config(n_gpus: int) -> dict:
    """The `config` object of the JSON line, the same for both arms."""
    return {"workload": WORKLOAD, "passes_per_step": PASSES_PER_STEP, "l2": L2_NOTE,
            "parallelism": "dp%d (independent batches, no collective)" % n_gpus}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index = index
        self.samples = []
        self.proc = None

    def run(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) >= 6:
                    self.samples.append(parts)
        except Exception:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        sm, smax, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0]))
                smax = max(smax, float(s[1]))
            except ValueError:
                continue
            for name, val in zip(names, s[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # only the busiest half of the samples is "under load" (the sampler also sees idle gaps)
        sm_sorted = sorted(sm)
        under = sm_sorted[len(sm_sorted) // 2:] if sm_sorted else []
        return {"sm_mhz": statistics.median(under) if under else None, "sm_max_mhz": smax or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------ CPU oracle legs

def oracle_sample_seconds(sample_rows: int = 256):
    """Time the oracle, as it stands, on a bounded sample of the step and scale to a full step.

    Cast: `sample_rows` rows of each tensor in both orientations (all host threads, row slabs).
    GEMM: `sample_rows` output rows of each product in FP64 over decoded operands (numpy/BLAS).
    Returns (seconds for the sample, estimated seconds for the full step, description).
    """
    import numpy as np
    import oracle as orc
    from paper_2506_08027_b200 import synth

    threads = os.cpu_count() or 1
    r = sample_rows
    x = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.gaussian((r, H), synth.seed_for(2, 0))))
    w = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.gaussian((r, H), synth.seed_for(2, 1), 0.02)))
    dy = synth.bf16_bits_as_f32(synth.f32_to_bf16_bits(synth.output_gradient((r, F), synth.seed_for(2, 2))))
    t0 = time.perf_counter()
    q = {}
    for name, t in (("x", x), ("w", w), ("dy", dy)):
        q[name, "r"] = orc.quantize_threads(t, orc.ROW, orc.RULE_PAPER, orc.E4M3, threads)
        q[name, "c"] = orc.quantize_threads(t, orc.COL, orc.RULE_PAPER, orc.E4M3, threads)
    t_cast = time.perf_counter() - t0
    cast_full = t_cast * (T * H + F * H + T * F) / float(r * H + r * H + r * F)
    # the same conversion on ONE thread (256 rows of dY, both orientations): the oracle's scalar rate
    one = dy[:min(r, 256)]
    t1 = time.perf_counter()
    orc.quantize(one, orc.ROW, orc.RULE_PAPER, orc.E4M3)
    orc.quantize(one, orc.COL, orc.RULE_PAPER, orc.E4M3)
    t_one = time.perf_counter() - t1
    cast_gbs_one_thread = one.size * (2 + 2 * (1 + 1 / 32)) / t_one / 1e9
    t0 = time.perf_counter()
    if r == T:
        # the whole step: all three products in FP64 over the decoded operands (+ the |A||B| bound products)
        orc.gemm_f64(q["x", "r"][0], q["x", "r"][1], q["w", "r"][0], q["w", "r"][1], "k", "k")            # fprop
        orc.gemm_f64(q["dy", "r"][0], q["dy", "r"][1], q["w", "c"][0], q["w", "c"][1], "k", "mn")         # dgrad
        orc.gemm_f64(q["dy", "c"][0], q["dy", "c"][1], q["x", "c"][0], q["x", "c"][1], "mn", "mn")        # wgrad
        t_gemm = time.perf_counter() - t0
        gemm_full = t_gemm
        desc = ("the whole pass on the host: X, W, dY quantized in both orientations on %d threads (row slabs), then "
                "fprop, dgrad, wgrad as FP64 products of the decoded operands (+ the |A||B| bound products) via numpy" % threads)
    else:
        # GEMM sample: r x r outputs of fprop over the full K = H (decoded FP64 operands, two products)
        orc.gemm_f64(q["x", "r"][0], q["x", "r"][1], q["w", "r"][0], q["w", "r"][1])
        t_gemm = time.perf_counter() - t0
        gemm_full = t_gemm * STEP_FLOP / (2.0 * r * r * H)
        desc = ("%d rows of X, W, dY quantized in both orientations on %d threads; %dx%dx%d FP64 product "
                "(+|A||B| bound product) via numpy; scaled linearly to the full step" % (r, threads, r, r, H))
    oracle_sample_seconds.split = {   # the two halves of the metric for the oracle (same byte and FLOP counts as the GPU arm)
        "cast_gbs": CAST_BYTES / cast_full / 1e9, "cast_gbs_one_thread": cast_gbs_one_thread, "gemm_tflops": STEP_FLOP / gemm_full / 1e12,
        "cast_seconds_full_step": cast_full, "gemm_seconds_full_step": gemm_full}
    return t_cast + t_gemm, cast_full + gemm_full, desc, threads


def run_reference(args):
    """The CPU oracle as it stands, timed on the host cores: every step is ONE whole pass of the workload
    (all casts on all threads, the three products in FP64 through numpy), i.e. one of the PASSES_PER_STEP
    micro-batches that a step of the GPU arm holds; the rate is per pass either way."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(max(0, min(args.warmup, 1))):
        oracle_sample_seconds(256)
    times = []
    desc, threads = "", 1
    for _ in range(args.steps):
        _, sec_pass, desc, threads = oracle_sample_seconds(T)     # casts + products; drawing the inputs is not timed
        times.append(sec_pass)
    sec = statistics.mean(times)
    value = STEP_FLOP / sec / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": bench_config(args.gpus),
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                         "sample": "each step: one of the %d passes of a step, whole -- %s" % (PASSES_PER_STEP, desc),
                         "median_seconds_per_pass": statistics.median(times), "best_seconds_per_pass": min(times)},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ GPU arm

def max_over_ranks(ms: float, world: int, device) -> float:
    """Device time of the slowest rank (the job finishes when the last rank does)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, ms_step: float) -> float:
    """TFLOP/s of the whole job: every rank runs the same passes on its own batches (weak scaling).
    ms_step is the time of ONE pass."""
    return world * STEP_FLOP / (ms_step * 1e-3) / 1e12


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()  # fail loudly if the CUDA library is missing

    dev = "cuda"
    # each rank draws its own batch (data parallel: per-GPU work is fixed, no exchange on the path)
    X = synth.device_tensor("activation", (T, H), synth.seed_for(2, 0) + 1000 * rank)
    W = synth.device_tensor("weight", (F, H), synth.seed_for(2, 1))
    dY = synth.device_tensor("output_gradient", (T, F), synth.seed_for(2, 2) + 1000 * rank)
    qX = B.alloc_quantize_outputs(T, H, B.BOTH, B.SF_SWIZZLED)
    qW = B.alloc_quantize_outputs(F, H, B.BOTH, B.SF_SWIZZLED)
    qdY = B.alloc_quantize_outputs(T, F, B.BOTH, B.SF_SWIZZLED)
    Y = torch.empty((T, F), dtype=torch.bfloat16, device=dev)
    dX = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    dW = torch.empty((F, H), dtype=torch.bfloat16, device=dev)
    P, E, S = B.RULE_PAPER, B.E4M3, B.SF_SWIZZLED

    # the three casts of the step go out as one launch (one ramp-up and one tail instead of three)
    items = B.make_quantize_items([(X,) + qX, (W,) + qW, (dY,) + qdY])

    # ... and so do the three GEMMs, independent once the copies exist (one pool of tiles, no partly idle last waves)
    gemms = B.make_gemm_problems([
        (qX[0], qX[1], qW[0], qW[1], T, F, H, B.K_MAJOR, B.K_MAJOR, E, E, Y),          # fprop
        (qdY[0], qdY[1], qW[2], qW[3], T, H, F, B.K_MAJOR, B.MN_MAJOR, E, E, dX),       # dgrad
        (qdY[2], qdY[3], qX[2], qX[3], F, H, T, B.MN_MAJOR, B.MN_MAJOR, E, E, dW),      # wgrad
    ])

    def one_pass():
        B.mxfp8_quantize_multi(items, B.BF16, B.BOTH, P, E, S)
        B.mxfp8_gemm_multi(gemms, B.BF16)

    def step():
        for _ in range(PASSES_PER_STEP):
            one_pass()

    def passes_with_events(n):
        """n passes with an event before and after each of the two launches -> (cast ms, gemm ms, pass ms) lists."""
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
        for k in range(n):
            ev[k][0].record(); B.mxfp8_quantize_multi(items, B.BF16, B.BOTH, P, E, S)
            ev[k][1].record(); B.mxfp8_gemm_multi(gemms, B.BF16)
            ev[k][2].record()
        torch.cuda.synchronize()
        return ([e[0].elapsed_time(e[1]) for e in ev], [e[1].elapsed_time(e[2]) for e in ev],
                [e[0].elapsed_time(e[2]) for e in ev])

    def step_by_kernel(ev):
        # the same work with one launch per GEMM and an event before every launch: per-kernel durations
        ev[0].record(); B.mxfp8_quantize_multi(items, B.BF16, B.BOTH, P, E, S)
        ev[1].record(); B.mxfp8_gemm(qX[0], qX[1], qW[0], qW[1], T, F, H, B.K_MAJOR, B.K_MAJOR, E, E, Y)
        ev[2].record(); B.mxfp8_gemm(qdY[0], qdY[1], qW[2], qW[3], T, H, F, B.K_MAJOR, B.MN_MAJOR, E, E, dX)
        ev[3].record(); B.mxfp8_gemm(qdY[2], qdY[3], qX[2], qX[3], F, H, T, B.MN_MAJOR, B.MN_MAJOR, E, E, dW)
        ev[4].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- burst figure: the first 20 passes after an idle gap (boost clock, before the power cap bites)
    for _ in range(3):
        one_pass()
    step_by_kernel([torch.cuda.Event(enable_timing=True) for _ in range(5)])      # first use of the single-product kernels
    barrier()
    time.sleep(0.5)
    b_cast, b_gemm, b_pass = passes_with_events(20)
    burst_clock_mhz, _ = B.mxfp8_gemm_last_clock()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    if B.mxfp8_device_status() != 0:
        raise SystemExit("device status word reports a timeout during warm-up")

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)

    # ---- timed region 1: K steps of PASSES_PER_STEP passes, device time, max over ranks (no events inside)
    launches0 = B.mxfp8_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    launches = B.mxfp8_launch_count() - launches0
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    ms_step = ms_total / args.steps
    ms_pass = ms_step / PASSES_PER_STEP
    # the SM clock the last GEMM launch of the timed region really ran at (cycles / nanoseconds read inside the kernel)
    gemm_clock_mhz, gemm_probe_us = B.mxfp8_gemm_last_clock()

    # ---- timed region 2 (continues the steady state): per-launch events on every pass of a few more steps
    n_ev = PASSES_PER_STEP * max(1, min(args.steps, 8))
    s_cast, s_gemm, s_pass = passes_with_events(n_ev)
    steady_clock_mhz, _ = B.mxfp8_gemm_last_clock()
    cast_ms = statistics.median(s_cast)
    gemm_multi_ms = statistics.median(s_gemm)
    # ---- the yardstick in the same place: a plain device-to-device copy that moves as many bytes as the cast does
    # (half of them read, half written), launched where the cast is, in the same power state.  The measured copy rate of
    # MEASURED_PEAKS.json is taken alone at the boost clock; behind the GEMM launch the memory system's clients run at
    # the clock the power cap leaves, and this says how much of the cast's distance to that peak is the place it runs in.
    copy_src = torch.empty(int(CAST_BYTES) // 2, dtype=torch.uint8, device=dev)
    copy_dst = torch.empty_like(copy_src)
    cev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(PASSES_PER_STEP)]
    for k in range(PASSES_PER_STEP):
        cev[k][0].record(); copy_dst.copy_(copy_src)
        cev[k][1].record(); B.mxfp8_gemm_multi(gemms, B.BF16)
    torch.cuda.synchronize()
    copy_in_pass_ms = statistics.median(e[0].elapsed_time(e[1]) for e in cev)
    del copy_src, copy_dst
    # ---- timed region 3: the three GEMMs launched one by one (per-product breakdown)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(PASSES_PER_STEP)]
    for k in range(PASSES_PER_STEP):
        step_by_kernel(evs[k])
    torch.cuda.synchronize()
    dur = [[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs]
    gemm_ms = dict(zip(("fprop", "dgrad", "wgrad"), (statistics.median(d[i] for d in dur) for i in (1, 2, 3))))
    status = B.mxfp8_device_status()

    # ---- end to end through the host-buffer C-ABI call (pinned host memory, copies inside)
    e2e = None
    if not args.no_e2e:
        hx, hw, hdy = (t.cpu().pin_memory() for t in (X, W, dY))
        hy = torch.empty((T, F), dtype=torch.bfloat16).pin_memory()
        hdx = torch.empty((T, H), dtype=torch.bfloat16).pin_memory()
        hdw = torch.empty((F, H), dtype=torch.bfloat16).pin_memory()
        ws = torch.empty(B.mxfp8_linear_host_ws_bytes(T, H, F), dtype=torch.uint8, device=dev)
        B.mxfp8_linear_host(hx, hw, hdy, P, hy, hdx, hdw, ws)
        n_e2e = PASSES_PER_STEP                      # one step of the end-to-end path (about a third of a second)
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(n_e2e):
            B.mxfp8_linear_host(hx, hw, hdy, P, hy, hdx, hdw, ws)
        g1.record()
        barrier()
        e2e_ms = max_over_ranks(g0.elapsed_time(g1) / n_e2e, world, dev)     # per pass
        assert torch.equal(hy.cuda(), Y), "host-buffer path and device path disagree"
        e2e = {"value": whole_job_value(world, e2e_ms), "unit": "TFLOP/s", "ms_per_step": e2e_ms * PASSES_PER_STEP,
               "ms_per_pass": e2e_ms,
               "h2d_bytes_per_step": (T * H + F * H + T * F) * 2 * PASSES_PER_STEP,
               "d2h_bytes_per_step": (T * F + T * H + F * H) * 2 * PASSES_PER_STEP,
               "steps": 1, "passes": n_e2e}
        del ws

    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["sm_mhz_inside_gemm_kernel"] = round(gemm_clock_mhz, 1)
        clocks["sm_mhz_inside_gemm_kernel_burst"] = round(burst_clock_mhz, 1)
        clocks["note"] = ("sm_mhz is the driver's sampled clock (20 ms per sample); sm_mhz_inside_gemm_kernel is SM cycles / wall time read "
                          "by the last GEMM launch of the timed region itself (%.0f us alive), ..._burst the same for the 20th pass after an "
                          "idle gap" % gemm_probe_us)
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    fp8_burst = 2.0 * peaks["bf16_tflops"]                     # FP8 = 2x the BF16 tensor rate (Table 1)
    fp8_sustained = 2.0 * peaks["bf16_tflops_sustained"]
    gemm_tflops = {k: 2.0 * m * n * kk / (gemm_ms[k] * 1e-3) / 1e12 for k, (m, n, kk) in GEMM_SHAPES.items()}
    gemm_all = STEP_FLOP / (sum(gemm_ms.values()) * 1e-3) / 1e12
    cast_gbs = CAST_BYTES / (cast_ms * 1e-3) / 1e9
    gemm_multi_tflops = STEP_FLOP / (gemm_multi_ms * 1e-3) / 1e12    # the launch the timed passes use: all three products
    value = whole_job_value(world, ms_pass)

    def tf(ms):
        return STEP_FLOP / (ms * 1e-3) / 1e12

    def gbs(ms):
        return CAST_BYTES / (ms * 1e-3) / 1e9

    b_gemm_ms, b_cast_ms = statistics.median(b_gemm), statistics.median(b_cast)
    burst = {"passes": len(b_pass), "after_idle_s": 0.5, "ms_per_pass": statistics.median(b_pass), "best_ms_per_pass": min(b_pass),
             "value": tf(statistics.median(b_pass)), "gemm_tflops": tf(b_gemm_ms), "gemm_ms": b_gemm_ms,
             "gemm_frac_of_2x_bf16_burst": tf(b_gemm_ms) / fp8_burst, "cast_gbs": gbs(b_cast_ms), "cast_ms": b_cast_ms,
             "cast_frac_of_measured_copy": gbs(b_cast_ms) / peaks["hbm_gbs"], "sm_mhz_inside_gemm_kernel": round(burst_clock_mhz, 1),
             "gemm_mcycles": b_gemm_ms * burst_clock_mhz * 1e-3}
    steady = {"passes": len(s_pass), "ms_per_pass": statistics.median(s_pass), "best_ms_per_pass": min(s_pass),
              "value": tf(statistics.median(s_pass)), "gemm_tflops": gemm_multi_tflops, "gemm_ms": gemm_multi_ms,
              "gemm_best_ms": min(s_gemm), "gemm_frac_of_2x_bf16_sustained": gemm_multi_tflops / fp8_sustained,
              "cast_gbs": cast_gbs, "cast_ms": cast_ms, "cast_best_ms": min(s_cast),
              "sm_mhz_inside_gemm_kernel": round(steady_clock_mhz, 1), "gemm_mcycles": gemm_multi_ms * steady_clock_mhz * 1e-3,
              "note": "per-launch CUDA events on every pass, taken right after the timed region (same thermal and power state)"}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        s, f, desc, threads = oracle_sample_seconds(8192)
        cpu = {"value": STEP_FLOP / f / 1e12, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
               "sample": "one pass (one of the %d of a step) -- %s" % (PASSES_PER_STEP, desc), "sample_seconds": s,
               **getattr(oracle_sample_seconds, "split", {})}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "ms_per_pass": ms_pass, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "fp8_e4m3 x fp8_e4m3 -> f32 accumulate", "data": "synthetic",
        "config": bench_config(world),
        "cast": {"value": cast_gbs, "unit": "GB/s", "ms": cast_ms, "bytes": CAST_BYTES,
                 "frac_of_measured_copy": cast_gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": cast_gbs / NOMINAL_HBM_GBS},
        "gemm": {"value": gemm_multi_tflops, "unit": "TFLOP/s", "ms": gemm_multi_ms,
                 "frac_of_2x_measured_bf16_sustained": gemm_multi_tflops / fp8_sustained,
                 "frac_of_2x_measured_bf16_burst": gemm_multi_tflops / fp8_burst, "frac_of_nominal_4.5PF": gemm_multi_tflops / NOMINAL_FP8_TFLOPS,
                 "launched_one_by_one": {"value": gemm_all, "ms": gemm_ms, "tflops": gemm_tflops}},
        "burst": burst, "steady": steady,
        # the dominant kernel, timed inside the long steady-state run: against the sustained peak
        "roofline": {"bound": "tensor", "kernel": "gemm_kernel<256, pair, multi> (fprop + dgrad + wgrad in one launch)",
                     "achieved": gemm_multi_tflops, "peak": fp8_sustained, "unit": "TFLOP/s", "frac": gemm_multi_tflops / fp8_sustained,
                     "peak_source": "2 x %s bf16 sustained TFLOP/s (Table 1: MXFP8 = 2x BF16); steady state of a %.2f s timed region"
                                    % (peaks["source"], ms_total * 1e-3),
                     "algorithmic_flop_per_launch": STEP_FLOP, "sm_mhz_inside_kernel": round(steady_clock_mhz, 1),
                     "traffic": NCU_TRAFFIC_GEMM_MULTI, "traffic_note": "ncu capture of this launch, see profiles/"},
        # the same launch in the first 20 passes after an idle gap: against the burst peak
        "roofline_burst": {"bound": "tensor", "achieved": tf(b_gemm_ms), "peak": fp8_burst, "unit": "TFLOP/s",
                           "frac": tf(b_gemm_ms) / fp8_burst, "peak_source": "2 x %s bf16 burst TFLOP/s" % peaks["source"],
                           "sm_mhz_inside_kernel": round(burst_clock_mhz, 1)},
        "roofline_cast": {"bound": "hbm", "kernel": "quantize_tma_kernel<bf16,e4m3,row+col>", "achieved": cast_gbs,
                          "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": cast_gbs / peaks["hbm_gbs"],
                          "peak_source": peaks["source"], "algorithmic_bytes_per_element": 4.0625,
                          "algorithmic_bytes_per_launch": CAST_BYTES, "frac_burst": gbs(b_cast_ms) / peaks["hbm_gbs"],
                          "copy_of_the_same_bytes_in_the_pass_gbs": gbs(copy_in_pass_ms),
                          "frac_of_that_copy": cast_gbs / gbs(copy_in_pass_ms),
                          "copy_note": "a plain device-to-device copy of CAST_BYTES / 2 (read + written = the cast's bytes) launched in the cast's "
                                       "place, between the GEMM launches of the steady state; torch's copy_, a yardstick, not part of the path",
                          "traffic": NCU_TRAFFIC_QUANTIZE_STEP,
                          "traffic_note": "ncu capture of this launch (X, W, dY in one), see profiles/"},
        "e2e": e2e, "gpu_launches": int(launches), "device_status": status, "clocks": clocks,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_case(args):
    """One kernel on one small case, a few launches, nothing else: the target of ncu captures.
    quantize: BF16 8192x8192 in both orientations; gemm: the 8192x8192x2048 fprop product
    (gemm8k: 8192^3);
    dequantize: 8192x8192 row-blocked bytes to BF16; fake_quantize: the BF16 8192x8192 round trip,
    row blocks."""
    import torch
    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200 import synth
    torch.cuda.set_device(0)
    n = 8192
    P, E, S = B.RULE_PAPER, B.E4M3, B.SF_SWIZZLED
    x = synth.device_tensor("activation", (n, n), 1)
    q = B.alloc_quantize_outputs(n, n, B.BOTH, S)
    reps = max(1, args.steps)
    if args.case == "quantize":
        for _ in range(reps):
            B.mxfp8_quantize(x, B.BOTH, P, E, *q, S)
    elif args.case == "step":
        # the benchmark step's two launches: the batched cast of X, W, dY and the three GEMMs in one launch
        X = synth.device_tensor("activation", (T, H), 2)
        W = synth.device_tensor("weight", (F, H), 3)
        dY = synth.device_tensor("output_gradient", (T, F), 4)
        qs = [B.alloc_quantize_outputs(t.shape[0], t.shape[1], B.BOTH, S) for t in (X, W, dY)]
        items = B.make_quantize_items([(t,) + o for t, o in zip((X, W, dY), qs)])
        Y, dX, dW = (torch.empty(sh, dtype=torch.bfloat16, device="cuda") for sh in ((T, F), (T, H), (F, H)))
        qX, qW, qdY = qs
        gemms = B.make_gemm_problems([
            (qX[0], qX[1], qW[0], qW[1], T, F, H, B.K_MAJOR, B.K_MAJOR, E, E, Y),
            (qdY[0], qdY[1], qW[2], qW[3], T, H, F, B.K_MAJOR, B.MN_MAJOR, E, E, dX),
            (qdY[2], qdY[3], qX[2], qX[3], F, H, T, B.MN_MAJOR, B.MN_MAJOR, E, E, dW)])
        for _ in range(reps):
            B.mxfp8_quantize_multi(items, B.BF16, B.BOTH, P, E, S)
            B.mxfp8_gemm_multi(gemms, B.BF16)
    elif args.case == "grouped":
        # per-expert fprop of a 64-expert layer (hidden 2048, expert FFN 1408, 49152 routed tokens, uniform routing)
        import numpy as np
        Hd, Fe, G = 2048, 1408, 64
        rng = np.random.default_rng(2506)
        padded = (rng.multinomial(8192 * 6, np.full(G, 1.0 / G)) + 127) // 128 * 128
        offs = np.concatenate([[0], np.cumsum(padded)]).astype(np.int32)
        Tt = int(offs[-1])
        xa = synth.device_tensor("activation", (Tt, Hd), 21)
        wst = synth.device_tensor("weight", (G * Fe, Hd), 23)
        qx = B.alloc_quantize_outputs(Tt, Hd, B.ROW, S); B.mxfp8_quantize(xa, B.ROW, P, E, *qx, S)
        qw = B.alloc_quantize_outputs(G * Fe, Hd, B.ROW, S); B.mxfp8_quantize(wst, B.ROW, P, E, *qw, S)
        yg = torch.empty((Tt, Fe), dtype=torch.bfloat16, device="cuda")
        off_d = torch.from_numpy(offs).cuda()
        for _ in range(reps):
            B.mxfp8_grouped_gemm(qx[0], qx[1], qw[0], qw[1], off_d, B.GROUP_M, Tt, Fe, Hd, B.K_MAJOR, E, E, yg)
    elif args.case == "grouped_wgrad":
        # per-expert wgrad of the same layer: dW_g = dY_g^T X_g over the expert's tokens (both operands token-major)
        import numpy as np
        Hd, Fe, G = 2048, 1408, 64
        rng = np.random.default_rng(2506)
        padded = (rng.multinomial(8192 * 6, np.full(G, 1.0 / G)) + 127) // 128 * 128
        offs = np.concatenate([[0], np.cumsum(padded)]).astype(np.int32)
        Tt = int(offs[-1])
        xa = synth.device_tensor("activation", (Tt, Hd), 21)
        dya = synth.device_tensor("output_gradient", (Tt, Fe), 22)
        qx = B.alloc_quantize_outputs(Tt, Hd, B.COL, S); B.mxfp8_quantize(xa, B.COL, P, E, *qx, S)
        qdy = B.alloc_quantize_outputs(Tt, Fe, B.COL, S); B.mxfp8_quantize(dya, B.COL, P, E, *qdy, S)
        dwg = torch.empty((G * Fe, Hd), dtype=torch.bfloat16, device="cuda")
        off_d = torch.from_numpy(offs).cuda()
        for _ in range(reps):
            B.mxfp8_grouped_gemm(qdy[2], qdy[3], qx[2], qx[3], off_d, B.GROUP_K, Fe, Hd, Tt, B.MN_MAJOR, E, E, dwg)
    elif args.case == "scatter":
        # the WGRAD product of the benchmark layer, its FP32 result added into 8 owner buffers (all on this device)
        xs = synth.device_tensor("activation", (T, H), 2)
        dys = synth.device_tensor("output_gradient", (T, F), 3)
        qx = B.alloc_quantize_outputs(T, H, B.COL, S); B.mxfp8_quantize(xs, B.COL, P, E, *qx, S)
        qdy = B.alloc_quantize_outputs(T, F, B.COL, S); B.mxfp8_quantize(dys, B.COL, P, E, *qdy, S)
        dw32 = torch.zeros((F, H), dtype=torch.float32, device="cuda")
        ptrs = B.make_owner_pointers([dw32[r * (F // 8):] for r in range(8)])
        for _ in range(reps):
            B.mxfp8_gemm_reduce_scatter(qdy[2], qdy[3], qx[2], qx[3], F, H, T, B.MN_MAJOR, B.MN_MAJOR, E, E, ptrs, 3)
    elif args.case == "glu":
        # SwiGLU fused ahead of the conversion: source 8192 x (2 x 8192) BF16, both orientations
        src2 = synth.device_tensor("gaussian", (n, 2 * n), 13, "bf16")
        for _ in range(reps):
            B.mxfp8_glu_quantize(src2, B.ACT_SILU, B.BOTH, P, E, *q, S)
    elif args.case == "fake_quantize":
        dst = torch.empty_like(x)
        for _ in range(reps):
            B.mxfp8_fake_quantize(x, B.ROW, P, E, dst, None)
    elif args.case == "dequantize":
        B.mxfp8_quantize(x, B.BOTH, P, E, *q, S)
        dst = torch.empty_like(x)
        for _ in range(reps):
            B.mxfp8_dequantize(q[0], q[1], B.ROW, E, S, dst)
    else:
        m_, n_, k_ = (8192, 8192, 8192) if args.case == "gemm8k" else (T, F, H)
        a = synth.device_tensor("activation", (m_, k_), 2)
        w = synth.device_tensor("weight", (n_, k_), 3)
        qa = B.alloc_quantize_outputs(m_, k_, B.ROW, S)
        qw = B.alloc_quantize_outputs(n_, k_, B.ROW, S)
        B.mxfp8_quantize(a, B.ROW, P, E, *qa, S)
        B.mxfp8_quantize(w, B.ROW, P, E, *qw, S)
        y = torch.empty((m_, n_), dtype=torch.bfloat16, device="cuda")
        epi = None
        if args.case == "gemm_fused":        # the fprop product with the row + column MXFP8 output next to D
            keep = B.alloc_quantize_outputs(m_, n_, B.BOTH, S)
            epi = B.make_epilogue(B.BOTH, P, E, *keep)
        for _ in range(reps):
            B.mxfp8_gemm(qa[0], qa[1], qw[0], qw[1], m_, n_, k_, B.K_MAJOR, B.K_MAJOR, E, E, y, epi=epi)
    torch.cuda.synchronize()
    print(json.dumps({"case": args.case, "launches": int(B.mxfp8_launch_count()), "device_status": B.mxfp8_device_status()}))


def _time_calls(fn, n_bufs, min_iters=10, min_ms=30.0):
    """Average device time of fn(i) in ms (CUDA events), i cycling through n_bufs rotated buffers."""
    import torch
    for i in range(3):
        fn(i % n_bufs)
    torch.cuda.synchronize()
    iters = min_iters
    while True:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            fn(i % n_bufs)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if ms >= min_ms or iters >= 2000:
            return ms / iters
        iters *= 4


def _time_graph(fn, n_bufs, calls=20, replays=20):
    """Device time of fn(i) in ms with the host out of the picture: `calls` launches captured once in a CUDA graph,
    the graph replayed `replays` times between two events."""
    import torch
    for i in range(3):
        fn(i % n_bufs)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(calls):
            fn(i % n_bufs)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (calls * replays)


def run_sweep(args):
    """Tables for the cast sweep (sizes x shapes x dtypes x orientations) and the GEMM shape sweep
    (square sizes, the skinny wgrad, the 8B decoder-block GEMMs, with and without the fused MXFP8
    output).  Prints markdown; not part of the one-line contract."""
    import torch
    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200 import synth
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    P, S = B.RULE_PAPER, B.SF_SWIZZLED
    if args.sweep == "cast":
        # Config-4 sweep.  Part 1: sizes x shapes x dtypes x orientations, each shape with "its" distribution.
        # Part 2 (at 256 MB): every distribution on every shape, E5M2 beside E4M3 in every orientation; the
        # distribution with 0.01 % NaN / Inf sends the slabs that meet one through the careful path.
        # host us/call: wall time of the C-ABI call alone (argument checks, tensor maps, launch), 200 calls.
        def cell(dtype, esz, nbytes, cols, kind, orients, elems):
            rows = max(32, (nbytes // (cols * esz)) // 32 * 32)
            n_bufs = max(1, min(4, int((768 << 20) // (rows * cols * esz)) + 1)) if nbytes < (1 << 30) else 1
            srcs = [synth.device_tensor(kind, (rows, cols), 7 + i, dtype) for i in range(n_bufs)]
            for orient, oname in orients:
                for elem in elems:
                    outs = B.alloc_quantize_outputs(rows, cols, orient, S)
                    ms = _time_calls(lambda i: B.mxfp8_quantize(srcs[i], orient, P, elem, *outs, S), n_bufs)
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                    for i in range(200):
                        B.mxfp8_quantize(srcs[0], orient, P, elem, *outs, S)
                    host_us = (time.perf_counter() - t0) / 200 * 1e6 if nbytes <= (16 << 20) else float("nan")
                    torch.cuda.synchronize()
                    by = rows * cols * (esz + (2 if orient == B.BOTH else 1) * (1 + 1 / 32))
                    gbs = by / ms / 1e6
                    # the same launches replayed from a CUDA graph: what the kernel takes when the host is not the limit
                    graph = ""
                    if nbytes <= (64 << 20):
                        gms = _time_graph(lambda i: B.mxfp8_quantize(srcs[i], orient, P, elem, *outs, S), n_bufs)
                        graph = "%.1f us = %.2f" % (gms * 1e3, by / gms / 1e6 / peaks["hbm_gbs"])
                    print("| %s | %d MB | %d x %d | %s | %s | %s | %.1f | %.0f | %.2f | %s | %s |" % (
                        dtype, nbytes >> 20, rows, cols, kind, oname, "e4m3" if elem == B.E4M3 else "e5m2",
                        ms * 1e3, gbs, gbs / peaks["hbm_gbs"], "-" if host_us != host_us else "%.1f" % host_us, graph or "-"), flush=True)
                    del outs
            del srcs
            torch.cuda.empty_cache()

        all_o = ((B.ROW, "row"), (B.COL, "col"), (B.BOTH, "both"))
        own_kind = {4096: "gaussian", 14336: "gradient_like", 8288: "student_t"}
        print("| dtype | source bytes | rows x cols | dist | orient | elem | us | GB/s | of measured copy | host us/call | from a CUDA graph: us = of copy |")
        print("|---|---|---|---|---|---|---|---|---|---|---|")
        for dtype, esz in (("bf16", 2), ("fp32", 4)):
            for nbytes in (1 << 20, 4 << 20, 16 << 20, 64 << 20, 256 << 20, 1 << 30, 4 << 30):
                for cols in (4096, 14336, 8288):
                    if nbytes >= (1 << 30) and cols != 4096 and dtype == "fp32":
                        continue
                    cell(dtype, esz, nbytes, cols, own_kind[cols], all_o, (B.E4M3,))
        print()
        print("Every distribution on every shape, both element types, 256 MB sources:")
        print()
        print("| dtype | source bytes | rows x cols | dist | orient | elem | us | GB/s | of measured copy | host us/call | from a CUDA graph: us = of copy |")
        print("|---|---|---|---|---|---|---|---|---|---|---|")
        for dtype, esz in (("bf16", 2), ("fp32", 4)):
            for cols in (4096, 14336, 8288):
                for kind in ("gaussian", "student_t", "gradient_like", "nonfinite"):
                    cell(dtype, esz, 256 << 20, cols, kind, all_o if dtype == "bf16" else ((B.BOTH, "both"),), (B.E4M3, B.E5M2))
        return
    if args.sweep == "rules":
        # The comparison of Sec. 3.3 (the paragraph after Algorithm 1; Fig. 5's subject) on synthetic tensors: for each
        # distribution x source dtype x element type, the share of blocks whose scale differs between the paper's rule
        # and the OCP one, the share of finite elements that the OCP scale pushes beyond destmax (clamped by the
        # saturating cast; none under the paper's rule), and the relative Frobenius error of the MXFP8 round trip under
        # each rule -- all through mxfp8_quantize / mxfp8_fake_quantize on the GPU, with the oracle's figures for the
        # first 2^22 elements of the same tensor beside them.
        import numpy as np
        import oracle as orc
        rows, cols = 8192, 4096
        print("| dist | source | elem | blocks with different scales | oracle | elements clamped, OCP | oracle | clamped, paper | round-trip error, paper | oracle | round-trip error, OCP | oracle |")
        print("|---|---|---|---|---|---|---|---|---|---|---|---|")
        for kind in ("gaussian", "student_t", "gradient_like", "nonfinite"):
            for dtype in ("bf16", "fp32"):
                src = synth.device_tensor(kind, (rows, cols), 41, dtype)
                x = src.float()
                fin = torch.isfinite(x)
                x0 = torch.where(fin, x, torch.zeros_like(x)).double()
                norm = float(x0.pow(2).sum().sqrt())
                host = src[:1024].float().cpu().numpy()
                hfin = np.isfinite(host)
                h0 = np.where(hfin, host.astype(np.float64), 0.0)
                for elem, ename, destmax in ((B.E4M3, "e4m3", 448.0), (B.E5M2, "e5m2", 57344.0)):
                    res, ores = {}, {}
                    for rule, rname in ((B.RULE_PAPER, "paper"), (B.RULE_OCP, "ocp")):
                        q, sc, _, _ = B.alloc_quantize_outputs(rows, cols, B.ROW, B.SF_LINEAR)
                        B.mxfp8_quantize(src, B.ROW, rule, elem, q, sc, None, None, B.SF_LINEAR)
                        back = torch.empty_like(src)
                        B.mxfp8_fake_quantize(src, B.ROW, rule, elem, back, None)
                        scale = torch.exp2(sc.view(rows, cols // 32).double() - 127.0).repeat_interleave(32, dim=1)
                        res[rname] = {"s": sc.view(rows, cols // 32).clone(),
                                      "clamped": float(((x0.abs() / scale) > destmax).sum() / fin.sum()),
                                      "err": float(torch.where(fin, back.double() - x0, torch.zeros_like(x0)).pow(2).sum().sqrt()) / norm}
                        oq, osc = orc.quantize_threads(host, orc.ROW, rule, elem, os.cpu_count() or 1)
                        od = orc.dequantize_f64(oq, osc, orc.ROW, elem)
                        oscale = np.repeat(np.exp2(osc.astype(np.float64) - 127.0), 32, axis=1)
                        ores[rname] = {"s": osc, "clamped": float((np.abs(h0) / oscale > destmax).sum() / hfin.sum()),
                                       "err": float(np.sqrt((np.where(hfin, od - h0, 0.0) ** 2).sum() / (h0 ** 2).sum()))}
                        del q, sc, back
                    differ = float((res["paper"]["s"] != res["ocp"]["s"]).float().mean())
                    odiffer = float((ores["paper"]["s"] != ores["ocp"]["s"]).mean())
                    print("| %s | %s | %s | %.2f %% | %.2f %% | %.3f %% | %.3f %% | %.3f %% | %.4f | %.4f | %.4f | %.4f |" % (
                        kind, dtype, ename, 100 * differ, 100 * odiffer, 100 * res["ocp"]["clamped"], 100 * ores["ocp"]["clamped"],
                        100 * res["paper"]["clamped"], res["paper"]["err"], ores["paper"]["err"], res["ocp"]["err"], ores["ocp"]["err"]), flush=True)
        assert B.mxfp8_device_status() == 0
        return
    if args.sweep == "moe":
        # per-expert GEMMs of a mixture-of-experts FFN (App. A.4 trains a 16B-total / 2.5B-active model; the layer here
        # has that class's shape: hidden 2048, expert FFN 1408, 64 experts, 6 experts per token, 8192 tokens per batch).
        # Token counts per expert are multinomial, each expert's segment padded to a multiple of 128 rows.
        import numpy as np
        Hd, Fe, G, topk, tokens = 2048, 1408, 64, 6, 8192
        print("| case | experts | routed tokens (padded) | N | K | us | TFLOP/s | of 2x measured BF16 | dense GEMM of the same size: us |")
        print("|---|---|---|---|---|---|---|---|---|")
        for skew, label in ((0.0, "uniform routing"), (1.0, "skewed routing")):
            rng = np.random.default_rng(2506)
            w = np.exp(skew * rng.standard_normal(G))
            counts = rng.multinomial(tokens * topk, w / w.sum())
            padded = (counts + 127) // 128 * 128
            offs = np.concatenate([[0], np.cumsum(padded)]).astype(np.int32)
            Tt = int(offs[-1])
            off_d = torch.from_numpy(offs).cuda()
            x = synth.device_tensor("activation", (Tt, Hd), 21)
            dy = synth.device_tensor("output_gradient", (Tt, Fe), 22)
            wst = synth.device_tensor("weight", (G * Fe, Hd), 23)
            qx = B.alloc_quantize_outputs(Tt, Hd, B.BOTH, S); B.mxfp8_quantize(x, B.BOTH, P, B.E4M3, *qx, S)
            qdy = B.alloc_quantize_outputs(Tt, Fe, B.BOTH, S); B.mxfp8_quantize(dy, B.BOTH, P, B.E4M3, *qdy, S)
            qw = B.alloc_quantize_outputs(G * Fe, Hd, B.BOTH, S); B.mxfp8_quantize(wst, B.BOTH, P, B.E4M3, *qw, S)
            y = torch.empty((Tt, Fe), dtype=torch.bfloat16, device="cuda")
            dx = torch.empty((Tt, Hd), dtype=torch.bfloat16, device="cuda")
            dw = torch.empty((G * Fe, Hd), dtype=torch.bfloat16, device="cuda")
            cases = (
                ("fprop", lambda i: B.mxfp8_grouped_gemm(qx[0], qx[1], qw[0], qw[1], off_d, B.GROUP_M, Tt, Fe, Hd, B.K_MAJOR, B.E4M3, B.E4M3, y),
                 Fe, Hd, lambda i: B.mxfp8_gemm(qx[0], qx[1], qw[0], qw[1], Tt, Fe, Hd, B.K_MAJOR, B.K_MAJOR, B.E4M3, B.E4M3, y)),
                ("dgrad", lambda i: B.mxfp8_grouped_gemm(qdy[0], qdy[1], qw[2], qw[3], off_d, B.GROUP_M, Tt, Hd, Fe, B.MN_MAJOR, B.E4M3, B.E4M3, dx),
                 Hd, Fe, lambda i: B.mxfp8_gemm(qdy[0], qdy[1], qw[2], qw[3], Tt, Hd, Fe, B.K_MAJOR, B.MN_MAJOR, B.E4M3, B.E4M3, dx)),
                ("wgrad", lambda i: B.mxfp8_grouped_gemm(qdy[2], qdy[3], qx[2], qx[3], off_d, B.GROUP_K, Fe, Hd, Tt, B.MN_MAJOR, B.E4M3, B.E4M3, dw),
                 Hd, None, lambda i: B.mxfp8_gemm(qdy[2], qdy[3], qx[2], qx[3], Fe, Hd, Tt, B.MN_MAJOR, B.MN_MAJOR, B.E4M3, B.E4M3, dw[:Fe])),
            )
            for name, fn, n_, k_, dense in cases:
                ms = _time_calls(fn, 1)
                ms_dense = _time_calls(dense, 1)
                flop = 2.0 * Tt * Fe * Hd
                tf = flop / ms / 1e9
                print("| %s, %s | %d | %d (%d) | %d | %s | %.1f | %.0f | %.2f | %.1f |" % (
                    name, label, G, int(counts.sum()), Tt, n_, k_ if k_ else "tokens of the expert", ms * 1e3, tf,
                    tf / (2 * peaks["bf16_tflops"]), ms_dense * 1e3), flush=True)
            assert B.mxfp8_device_status() == 0
        return
    if args.sweep == "dp":
        # the data-parallel exchange kernels on ONE GPU (all owners' buffers on this device: the additions go to local
        # memory instead of NVLink, everything else is what a rank of a multi-GPU job launches)
        from paper_2506_08027_b200.dp import DataParallelLinear
        E, MN = B.E4M3, B.MN_MAJOR
        x = synth.device_tensor("activation", (T, H), 31)
        w = synth.device_tensor("weight", (F, H), 32)
        dy = synth.device_tensor("output_gradient", (T, F), 33)
        qx = B.alloc_quantize_outputs(T, H, B.COL, S); B.mxfp8_quantize(x, B.COL, P, E, *qx, S)
        qdy = B.alloc_quantize_outputs(T, F, B.COL, S); B.mxfp8_quantize(dy, B.COL, P, E, *qdy, S)
        dw32 = torch.zeros((F, H), dtype=torch.float32, device="cuda")
        print("| WGRAD %d x %d x %d (tokens), FP32 result | us | TFLOP/s | of 2x measured BF16 |" % (F, H, T))
        print("|---|---|---|---|")
        cases = [("mxfp8_gemm, result stored", lambda i: B.mxfp8_gemm(qdy[2], qdy[3], qx[2], qx[3], F, H, T, MN, MN, E, E, dw32))]
        for owners_n in (1, 2, 8):
            ptrs = B.make_owner_pointers([dw32[r * (F // owners_n):] for r in range(owners_n)])
            cases.append(("mxfp8_gemm_reduce_scatter, result added into %d owner buffer%s" % (owners_n, "" if owners_n == 1 else "s"),
                          lambda i, ptrs=ptrs: B.mxfp8_gemm_reduce_scatter(qdy[2], qdy[3], qx[2], qx[3], F, H, T, MN, MN, E, E, ptrs, len(ptrs) // 2)))
        for name, fn in cases:
            ms = _time_calls(fn, 1)
            tf = 2.0 * F * H * T / ms / 1e9
            print("| %s | %.1f | %.0f | %.2f |" % (name, ms * 1e3, tf, tf / (2 * peaks["bf16_tflops"])), flush=True)
        y = torch.empty((T, F), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
        dw = torch.empty((F, H), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
        layer = DataParallelLinear(T, H, F)
        print()
        print("| whole step, T %d, H %d, F %d, one rank | launches | us |" % (T, H, F))
        print("|---|---|---|")
        print("| mxfp8_linear (dW in BF16) | 2 | %.1f |" % (1e3 * _time_calls(lambda i: B.mxfp8_linear(x, w, dy, P, y, dx, dw, ws), 1)), flush=True)
        print("| DataParallelLinear.step (dW added into the FP32 shard, zeroed every step) | 5 + memset | %.1f |" % (
            1e3 * _time_calls(lambda i: layer.step(x, w, dy), 1)), flush=True)
        assert B.mxfp8_device_status() == 0
        return
    if args.sweep == "emu":
        # the MXFP8 round trip (Sec. 3.1): reads the source once, writes one same-dtype tensor per orientation
        print("| dtype | rows x cols | orient | us | GB/s | of measured copy |")
        print("|---|---|---|---|---|---|")
        for dtype, esz in (("bf16", 2), ("fp32", 4)):
            for rows, cols in ((2048, 4096), (8192, 8192), (16384, 14336)):
                src = synth.device_tensor("gaussian", (rows, cols), 11, dtype)
                dr, dc = torch.empty_like(src), torch.empty_like(src)
                for orient, oname in ((B.ROW, "row"), (B.COL, "col"), (B.BOTH, "both")):
                    ms = _time_calls(lambda i: B.mxfp8_fake_quantize(src, orient, P, B.E4M3, dr if orient & B.ROW else None,
                                                                       dc if orient & B.COL else None), 1)
                    gbs = rows * cols * esz * (3 if orient == B.BOTH else 2) / ms / 1e6
                    print("| %s | %d x %d | %s | %.1f | %.0f | %.2f |" % (dtype, rows, cols, oname, ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
                del src, dr, dc
                torch.cuda.empty_cache()
        # an activation fused ahead of the conversion (mxfp8_act_quantize): same bytes as the plain conversion
        print()
        print("| activation + conversion, BF16 16384 x 8192, both orientations | us | GB/s | of measured copy |")
        print("|---|---|---|---|")
        rows, cols = 16384, 8192
        src = synth.device_tensor("gaussian", (rows, cols), 12, "bf16")
        outs = B.alloc_quantize_outputs(rows, cols, B.BOTH, S)
        for act, name in ((B.ACT_NONE, "none (plain mxfp8_quantize path)"), (B.ACT_RELU, "relu"), (B.ACT_RELU2, "squared relu"),
                          (B.ACT_SILU, "silu"), (B.ACT_GELU_TANH, "gelu (tanh)")):
            ms = _time_calls(lambda i: B.mxfp8_act_quantize(src, act, B.BOTH, P, B.E4M3, *outs, S), 1)
            gbs = rows * cols * (2 + 2 * (1 + 1 / 32)) / ms / 1e6
            print("| %s | %.1f | %.0f | %.2f |" % (name, ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
        src2 = synth.device_tensor("gaussian", (rows, 2 * cols), 13, "bf16")
        for act, name in ((B.ACT_SILU, "gated silu (SwiGLU): source 16384 x 16384 = (gate | up)"), (B.ACT_RELU, "gated relu (ReGLU)")):
            ms = _time_calls(lambda i: B.mxfp8_glu_quantize(src2, act, B.BOTH, P, B.E4M3, *outs, S), 1)
            gbs = rows * cols * (4 + 2 * (1 + 1 / 32)) / ms / 1e6       # gate and up are read, one [rows, cols] result in both orientations written
            print("| %s | %.1f | %.0f | %.2f |" % (name, ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
        del src2
        dh = synth.device_tensor("output_gradient", (rows, cols), 14, "bf16")
        for act, name in ((B.ACT_RELU2, "backward of squared relu: 2 relu(z) * dh, two sources"), (B.ACT_SILU, "backward of silu: silu'(z) * dh, two sources")):
            ms = _time_calls(lambda i: B.mxfp8_act_grad_quantize(dh, src, act, B.BOTH, P, B.E4M3, *outs, S), 1)
            gbs = rows * cols * (4 + 2 * (1 + 1 / 32)) / ms / 1e6       # z and dh are read, one [rows, cols] result in both orientations written
            print("| %s | %.1f | %.0f | %.2f |" % (name, ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
        del dh
        gamma = torch.ones(cols, dtype=torch.bfloat16, device="cuda")
        rstd = torch.empty(rows, dtype=torch.float32, device="cuda")
        ms = _time_calls(lambda i: B.mxfp8_rmsnorm_quantize(src, gamma, 1e-5, rstd, B.BOTH, P, B.E4M3, *outs, S), 1)
        gbs = rows * cols * (2 + 2 + 2 * (1 + 1 / 32)) / ms / 1e6       # the source is read twice (statistics, conversion)
        print("| rms normalisation (statistics launch + fused conversion; source read twice) | %.1f | %.0f | %.2f |" % (
            ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
        beta = torch.zeros(cols, dtype=torch.bfloat16, device="cuda")
        mean = torch.empty(rows, dtype=torch.float32, device="cuda")
        ms = _time_calls(lambda i: B.mxfp8_layernorm_quantize(src, gamma, beta, 1e-5, mean, rstd, B.BOTH, P, B.E4M3, *outs, S), 1)
        gbs = rows * cols * (2 + 2 + 2 * (1 + 1 / 32)) / ms / 1e6       # the statistics launch reads each row twice, the second time from cache
        print("| layer normalisation (statistics launch + fused conversion; source read twice from memory) | %.1f | %.0f | %.2f |" % (
            ms * 1e3, gbs, gbs / peaks["hbm_gbs"]), flush=True)
        return
    shapes = [("square", n, n, n, 0, 0) for n in (1024, 2048, 4096, 8192, 16384)]
    shapes.append(("skinny wgrad", 4096, 4096, 65536, 1, 1))
    Tk = 16384
    for name, fin, fout in (("qkv", 4096, 6144), ("o", 4096, 4096), ("ffn_up", 4096, 28672), ("ffn_down", 14336, 4096)):
        shapes.append((name + " fprop", Tk, fout, fin, 0, 0))
        shapes.append((name + " dgrad", Tk, fin, fout, 0, 1))
        shapes.append((name + " wgrad", fout, fin, Tk, 1, 1))
    # every cell is timed in three rounds, the variants of one shape interleaved inside each round (the launch runs under
    # the board's power cap and the clock drifts by several percent between rounds): the median of the rounds is
    # reported, with the SM clock the kernel itself measured and the product of the two in cycles
    print("| case | M | N | K | majors | out | fused MX out | us (median of 3) | min | max | TFLOP/s | of 2x measured BF16 burst | SM MHz in kernel | Mcycles |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
    fp8_peak = 2.0 * peaks["bf16_tflops"]
    for name, M, N, K, am, bm in shapes:
        def operand(mn, k, major, seed):
            if major == 0:
                x = synth.device_tensor("gaussian", (mn, k), seed)
                o = B.alloc_quantize_outputs(mn, k, B.ROW, S)
                B.mxfp8_quantize(x, B.ROW, P, B.E4M3, *o, S)
                return o[0], o[1]
            x = synth.device_tensor("gaussian", (k, mn), seed)
            o = B.alloc_quantize_outputs(k, mn, B.COL, S)
            B.mxfp8_quantize(x, B.COL, P, B.E4M3, *o, S)
            return o[2], o[3]
        Aq, As = operand(M, K, am, 11)
        Bq, Bs = operand(N, K, bm, 12)
        cells = []
        for out_dt, oname in ((torch.bfloat16, "bf16"), (torch.float32, "fp32")):
            for epi_o in (0, B.ROW, B.BOTH):
                if epi_o and out_dt == torch.float32:
                    continue
                if epi_o == B.BOTH and name == "square" and M not in (4096, 8192):
                    continue
                D = torch.empty((M, N), dtype=out_dt, device="cuda")
                epi, keep = None, None
                if epi_o:
                    keep = B.alloc_quantize_outputs(M, N, epi_o, S)
                    epi = B.make_epilogue(epi_o, P, B.E4M3, *keep)
                cells.append({"out": oname, "epi": epi_o, "D": D, "epi_obj": epi, "keep": keep, "ms": [], "mhz": []})
        for _ in range(3):
            for c in cells:
                c["ms"].append(_time_calls(lambda i: B.mxfp8_gemm(Aq, As, Bq, Bs, M, N, K, am, bm, B.E4M3, B.E4M3, c["D"], epi=c["epi_obj"]), 1, 10, 20.0))
                c["mhz"].append(B.mxfp8_gemm_last_clock()[0])
        for c in cells:
            ms, mhz = statistics.median(c["ms"]), statistics.median(c["mhz"])
            tf = 2.0 * M * N * K / ms / 1e9
            print("| %s | %d | %d | %d | %s%s | %s | %s | %.1f | %.1f | %.1f | %.0f | %.2f | %.0f | %.2f |" % (
                name, M, N, K, "kn"[0] if am == 0 else "m", "k" if bm == 0 else "n", c["out"],
                {0: "-", B.ROW: "row", B.BOTH: "row+col"}[c["epi"]], ms * 1e3, min(c["ms"]) * 1e3, max(c["ms"]) * 1e3, tf, tf / fp8_peak,
                mhz, ms * mhz * 1e-3), flush=True)
        del cells, Aq, As, Bq, Bs
        torch.cuda.empty_cache()
    assert B.mxfp8_device_status() == 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--case", default=None, choices=["quantize", "dequantize", "fake_quantize", "gemm", "gemm8k", "gemm_fused", "step", "grouped", "grouped_wgrad", "glu", "scatter"],
                    help="run one kernel on one small case and exit (for profiler captures)")
    ap.add_argument("--sweep", default=None, choices=["cast", "gemm", "emu", "moe", "dp", "rules"],
                    help="print the cast-bandwidth, GEMM-shape or round-trip (emu) sweep as a markdown table and exit")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
