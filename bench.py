"""Benchmark of the structured contraction library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one call of the hot path on the headline workload: the bf16 matmul
C[4096,4096] = A[4096,4096] . B[4096,4096] with f32 accumulation and f32 output (the largest
point of the matmul sweep).  Rank 0 prints ONE JSON line.  The line also carries, under
"per_op", the GFLOP/s and roofline fraction of the other configured ops (f32 matmul, both
convolutions, the large and the skinny matmul), each timed the same way on fewer iterations.

Multi-GPU (torchrun, one process per GPU): the op has no exchange step, so each rank runs
the same workload on its own device ("weak" scaling, no data-path collective); the value is
all ranks' flops over the slowest rank's device time.

--impl reference times the CPU oracle (plain C loop nest, as it stands) on a bounded sample
of the same workload on the host cores.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

M = N = K = 4096
WORKLOAD = "matmul 4096x4096x4096, bf16 inputs uniform[-1,1), f32 accumulate and output (largest point of the matmul sweep)"
FLOPS_PER_STEP = 2.0 * M * N * K
N_SETS = 3            # rotating (A, B, C) sets: 3 x 128 MB > the 126 MB L2

# DRAM bytes per launch of the dominant kernel from the committed ncu capture; None when the
# kernel changed after the capture was taken.
NCU_TRAFFIC_BYTES = None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def gpu_operand(shape, seed, tid, dist, dtype):
    import numpy as np
    import torch
    from paper_2202_03293_b200 import inputs
    payload, _ = inputs.make(shape, seed, tid, dist, dtype)
    if dtype == "bf16":
        return torch.from_numpy(payload.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(payload).cuda()


def time_launches(fn, iters, warmup):
    """Average device time per call in ms, CUDA events on the current (launching) stream."""
    import torch
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_graph(calls, reps, warmup=3):
    """Average device time per call in ms with the calls captured once into a CUDA graph
    and replayed, so that host-side call overhead is outside the measurement."""
    import torch
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for c in calls[:2]:
            c()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for c in calls:
            c()
    for _ in range(warmup):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps / len(calls)


def op_specs(sg, seed):
    """The other configured ops: name -> (label, flops, compulsory bytes, dtype, make(set) -> buffers, call)."""
    import torch

    def mm(Mx, Nx, Kx, dtype, label):
        es = 2 if dtype == "bf16" else 4
        return (label, 2.0 * Mx * Nx * Kx, (Mx * Kx + Kx * Nx) * es + Mx * Nx * 4, dtype,
                lambda s: (gpu_operand((Mx, Kx), seed, 10 + s, "uniform", dtype),
                           gpu_operand((Kx, Nx), seed, 40 + s, "uniform", dtype), torch.empty(Mx, Nx, device="cuda")),
                lambda a, b, c: sg.sg_matmul(a, b, c))

    return {
        "matmul128_f32": mm(128, 128, 128, "f32", "matmul 128^3 f32 (config 1)"),
        "matmul4096_f32": mm(4096, 4096, 4096, "f32", "matmul 4096^3 f32 (sweep corner)"),
        "matmul4096_bf16": mm(4096, 4096, 4096, "bf16", "matmul 4096^3 bf16 (sweep corner)"),
        "matmul1024_bf16": mm(1024, 1024, 1024, "bf16", "matmul 1024^3 bf16 (sweep point)"),
        "matmul8192_bf16": mm(8192, 8192, 8192, "bf16", "matmul 8192^3 bf16 (config 5)"),
        "matmul_skinny_bf16": mm(16384, 64, 4096, "bf16", "matmul 16384x64x4096 bf16 (config 5, skinny)"),
        # conv1d config 3: N=32, W=1026, C=64, KW=3, F=128, f32
        "conv1d_c3": ("conv_1d_nwc_wcf 32x1026x64 * 3x64x128 f32 (config 3)", 2.0 * 32 * 1024 * 128 * 3 * 64,
                      (32 * 1026 * 64 + 3 * 64 * 128) * 4 + 32 * 1024 * 128 * 4, "f32",
                      lambda s: (gpu_operand((32, 1026, 64), seed, 70 + s, "uniform", "f32"),
                                 gpu_operand((3, 64, 128), seed, 90, "uniform", "f32"),
                                 torch.empty(32, 1024, 128, device="cuda")),
                      lambda i, k, o: sg.sg_conv1d_nwc_wcf(i, k, o)),
        # conv2d config 4: N=16, 58x58x64, 3x3, F=128, bf16
        "conv2d_c4": ("conv_2d_nhwc_hwcf 16x58x58x64 * 3x3x64x128 bf16 (config 4)", 2.0 * 16 * 56 * 56 * 128 * 9 * 64,
                      (16 * 58 * 58 * 64 + 9 * 64 * 128) * 2 + 16 * 56 * 56 * 128 * 4, "bf16",
                      lambda s: (gpu_operand((16, 58, 58, 64), seed, 100 + s, "normal", "bf16"),
                                 gpu_operand((3, 3, 64, 128), seed, 120, "normal", "bf16"),
                                 torch.empty(16, 56, 56, 128, device="cuda")),
                      lambda i, k, o: sg.sg_conv2d_nhwc_hwcf(i, k, o)),
    }


def measure_op(sg, peaks, spec, reps=None):
    """Times one op: buffers rotate over enough sets to exceed L2 between reuses."""
    import torch
    label, flops, bytes_, dtype, make, call = spec
    ffma_peak = 148 * 128 * 2 * 1.965e9 / 1e12      # TFLOP/s at the maximum SM clock
    sets = min(16, max(2, int(400e6 // max(bytes_, 1)) + 1))
    bufs = [make(s) for s in range(sets)]
    ncalls = sets * 2 if bytes_ < 100e6 else sets
    calls = [(lambda b=bufs[i % sets]: call(*b)) for i in range(ncalls)]
    call(*bufs[0])
    torch.cuda.synchronize()
    fam = sg.sg_last_kernel()
    est_ms = max(flops / 3e14, 5e-3)
    if reps is None:
        reps = int(max(3, min(50, 0.25 / (est_ms * 1e-3 * ncalls))))
    ms = time_graph(calls, reps)
    host_ms = time_launches(lambda i: call(*bufs[i % sets]), max(3, min(100, ncalls * 2)), 2)
    tf = flops / (ms * 1e-3) / 1e12
    t_compute = flops / ((peaks["bf16_tflops"] if fam == sg.SG_KERNEL_TENSOR else ffma_peak) * 1e12)
    t_bytes = bytes_ / (peaks["hbm_gbs"] * 1e9)
    bound = max(t_compute, t_bytes)
    row = {"op": label, "dtype": dtype, "kernel": "tensor" if fam == sg.SG_KERNEL_TENSOR else "ffma",
           "us": round(ms * 1e3, 2), "us_with_host_call": round(host_ms * 1e3, 2), "gflops": round(tf * 1e3, 1),
           "gbs": round(bytes_ / (ms * 1e-3) / 1e9, 1),
           "bound": "hbm" if t_bytes > t_compute else ("tensor" if fam == sg.SG_KERNEL_TENSOR else "ffma"),
           "roofline_us": round(bound * 1e6, 2), "frac": round(bound / (ms * 1e-3), 4), "rotating_sets": sets,
           "timing": "CUDA graph replay"}
    del bufs, calls
    torch.cuda.empty_cache()
    return row


def per_op_table(sg, peaks, seed):
    specs = op_specs(sg, seed)
    return [measure_op(sg, peaks, specs[name]) for name in specs if name != "matmul4096_bf16"]


def cpu_baseline(target_seconds=12.0):
    """Times the oracle on a bounded sample (leading rows of the 4096^3 matmul) on the host cores."""
    from oracle import ref
    from paper_2202_03293_b200 import inputs
    seed = inputs.BASE_SEED + 1
    _, b = inputs.make((K, N), seed, 2, "uniform", "bf16")
    threads = ref.max_threads()
    rows = threads
    _, a = inputs.make((rows, K), seed, 1, "uniform", "bf16")
    t0 = time.perf_counter()
    ref.matmul(a, b)
    dt = time.perf_counter() - t0
    rows_full = int(min(M, max(rows, rows * target_seconds / max(dt, 1e-6))))
    rows_full -= rows_full % threads
    rows_full = max(rows_full, threads)
    _, a = inputs.make((rows_full, K), seed, 1, "uniform", "bf16")
    t0 = time.perf_counter()
    ref.matmul(a, b)
    dt = time.perf_counter() - t0
    gflops = 2.0 * rows_full * N * K / dt / 1e9
    return {"value": round(gflops, 3), "unit": "GFLOP/s", "cores": threads, "kind": "oracle",
            "sample": f"first {rows_full} of {M} rows of the 4096^3 matmul ({dt:.1f} s)"}, dt, rows_full


def run_reference(args, rank):
    if rank != 0:
        return
    vals = []
    info = None
    for i in range(args.warmup + args.steps):
        info, dt, rows = cpu_baseline(target_seconds=max(2.0, 60.0 / max(1, args.warmup + args.steps)))
        if i >= args.warmup:
            vals.append(info["value"])
    value = statistics.mean(vals)
    info["value"] = round(value, 3)
    line = {"impl": "reference", "metric": "matmul GFLOP/s (4096^3 bf16-valued inputs, f64 CPU oracle)", "value": round(value, 3),
            "unit": "GFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(FLOPS_PER_STEP / (value * 1e9) * 1e3, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD},
            "cpu_baseline": info, "e2e": {"value": round(value, 3), "unit": "GFLOP/s", "h2d_bytes_per_step": 0,
                                           "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-op", action="store_true", help="skip the per-op table")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--op", default=None, help="time only this op of the per-op table (used for profiler captures)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2202_03293_b200 import binding as sg
    from paper_2202_03293_b200 import inputs, sharding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sg.lib()
    peaks = load_peaks()
    seed = inputs.BASE_SEED + 1
    warmup = max(args.warmup, 3)

    if args.op is not None:
        specs = op_specs(sg, seed)
        if args.op not in specs:
            raise SystemExit(f"--op must be one of {sorted(specs)}")
        print(json.dumps(measure_op(sg, peaks, specs[args.op], reps=max(1, min(args.steps, 5)))), flush=True)
        return

    sets = [(gpu_operand((M, K), seed, 1 + 3 * s, "uniform", "bf16"), gpu_operand((K, N), seed, 2 + 3 * s, "uniform", "bf16"),
             torch.empty(M, N, device="cuda")) for s in range(N_SETS)]

    def step(i):
        a, b, c = sets[i % N_SETS]
        sg.sg_matmul(a, b, c)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = sg.sg_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    barrier()
    launches = sg.sg_launch_count() - launches0
    clocks = sampler.stop()
    sg.sg_check()
    ms_total = sharding.max_over_ranks(e0.elapsed_time(e1), device="cuda")
    ms_per_step = ms_total / args.steps
    value = world * FLOPS_PER_STEP / (ms_per_step * 1e-3) / 1e9      # GFLOP/s, all ranks

    # ---- end to end through the public call, host buffers, copies inside the timed region ----
    a_h = sets[0][0].cpu().pin_memory()
    b_h = sets[0][1].cpu().pin_memory()
    c_h = torch.empty(M, N).pin_memory()
    e2e_steps = max(3, min(20, args.steps))

    def e2e_step(i):
        a, b, c = sets[i % N_SETS]
        a.copy_(a_h, non_blocking=True)
        b.copy_(b_h, non_blocking=True)
        sg.sg_matmul(a, b, c)
        c_h.copy_(c, non_blocking=True)

    for i in range(3):
        e2e_step(i)
    barrier()
    e0.record()
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_ms = sharding.max_over_ranks(e0.elapsed_time(e1), device="cuda")
    e2e_value = world * FLOPS_PER_STEP / (e2e_ms / e2e_steps * 1e-3) / 1e9

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # the timed loop is one kernel launch per step, so the kernel's average duration is the
    # step time measured above (CUDA events on the launching stream)
    timed_seconds = ms_total * 1e-3
    peak_kind = "bf16_tflops_sustained" if timed_seconds >= 1.0 else "bf16_tflops"
    achieved_tf = FLOPS_PER_STEP / (ms_per_step * 1e-3) / 1e12
    roofline = {"bound": "tensor", "achieved": round(achieved_tf, 1), "peak": peaks[peak_kind], "unit": "TFLOP/s",
                "frac": round(achieved_tf / peaks[peak_kind], 4), "traffic": NCU_TRAFFIC_BYTES,
                "peak_source": f"{peaks['source']} {peak_kind} (timed region {timed_seconds:.2f} s)",
                "kernel": "tc_gemm_kernel", "algorithmic_flops_per_launch": FLOPS_PER_STEP,
                "frac_of_burst": round(achieved_tf / peaks["bf16_tflops"], 4),
                "frac_of_sustained": round(achieved_tf / peaks["bf16_tflops_sustained"], 4)}

    line = {"metric": "matmul GFLOP/s (and fraction of the tensor-core roofline) on B200", "value": round(value, 1),
            "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "N": N, "K": K,
                       "l2": f"inputs rotate over {N_SETS} buffer sets ({N_SETS * 128} MB) > 126 MB L2",
                       "parallelism": f"replicas x{world}, no collective"},
            "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": round(e2e_value, 1), "unit": "GFLOP/s", "h2d_bytes_per_step": 2 * M * K * 2,
                    "d2h_bytes_per_step": M * N * 4, "steps": e2e_steps}}
    if not args.no_per_op:
        del sets
        torch.cuda.empty_cache()
        line["per_op"] = per_op_table(sg, peaks, seed)
    if not args.no_cpu and world == 1:
        line["cpu_baseline"] = cpu_baseline()[0]
    elif world > 1:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
