"""Benchmark of the structured contraction library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass over the matmul sweep: C[M,N] = A[M,K] . B[K,N] for every M, N, K in
{256, 512, 1024, 2048, 4096} (125 shapes), once with bf16 inputs and once with f32 inputs, f32
accumulation and f32 output: 250 calls of sg_matmul on dense row-major buffers that stay
resident in HBM (6.3 GB, far beyond the L2).  Rank 0 prints ONE JSON line.  Its "roofline"
object describes the kernel that takes most of the step (the f32 tensor-core kernel); "per_op"
lists the other configured ops (the sweep's 4096^3 corner in both dtypes, config 1, both
convolutions, the large and the skinny matmul), each timed on its own by CUDA-graph replay.

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

SWEEP = (256, 512, 1024, 2048, 4096)
SHAPES = [(m, n, k) for m in SWEEP for n in SWEEP for k in SWEEP]
M = N = K = 4096          # the sweep's largest point (CPU sample, per-op table)
WORKLOAD = ("matmul sweep M,N,K in {256,512,1024,2048,4096} (125 shapes), bf16 inputs and again f32 inputs, "
            "uniform[-1,1), f32 accumulate and output")
FLOPS_PER_DTYPE = sum(2.0 * m * n * k for m, n, k in SHAPES)
FLOPS_PER_STEP = 2 * FLOPS_PER_DTYPE

METRIC = "matmul sweep GFLOP/s"      # the same string in both arms (ours and --impl reference)
UNIT = "GFLOP/s"
# tf32 : bf16 dense tensor throughput (nominal 1.1 : 2.25 PFLOP/s; the issue rate measured on
# this chip is exactly half)
TF32_OVER_BF16 = 0.5
NOMINAL_BF16_TFLOPS = 2250.0         # the chip's dense bf16 tensor rate as NVIDIA states it; tf32 is half of it
SAMPLES = 100                        # timing protocol of the paper's Section 4.3: 100 measurements, median and quartiles
# DRAM traffic of the dominant kernel: written next to the ncu summary it was read from, with a hash of the
# kernel's source files at capture time; None when the file is absent or the sources changed since
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "tc_gemm_f32_traffic.txt")
KERNEL_SOURCES = ("paper_2202_03293_b200/csrc/sg_tc.cu", "paper_2202_03293_b200/csrc/sg_tc_ptx.cuh")


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def traffic_per_launch(avg_algorithmic_bytes):
    """DRAM bytes per launch of the f32 tensor-core kernel, from one small ncu capture of a single shape scaled by
    algorithmic bytes to the step's average launch.  (bytes or None, note)."""
    if not os.path.exists(TRAFFIC_FILE):
        return None, "no capture on file"
    kv = {}
    with open(TRAFFIC_FILE) as f:
        for line in f:
            if ":" in line and not line.lstrip().startswith("#"):
                k, v = line.split(":", 1)
                kv[k.strip()] = v.strip()
    try:
        if kv["source_hash"] != kernel_source_hash():
            return None, "kernel sources changed since the capture"
        scale = avg_algorithmic_bytes / float(kv["algorithmic_bytes_of_captured_launch"])
        return round(float(kv["dram_bytes_per_launch"]) * scale), f"{kv.get('shape', '?')} captured, scaled by algorithmic bytes x{scale:.3f}"
    except (KeyError, ValueError):
        return None, "capture file unreadable"


def quartiles(xs):
    """median, p25, p75, mean of a list of samples."""
    xs = sorted(xs)
    q = statistics.quantiles(xs, n=4, method="inclusive") if len(xs) > 1 else [xs[0]] * 3
    return {"median": q[1], "p25": q[0], "p75": q[2], "mean": statistics.fmean(xs), "n": len(xs)}
BW_ROWS, BW_COLS = 16384, 12288   # shape of the memory-bound 2-D kernels' rows in the per-op table (805 MB of f32)


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


def time_graph(calls, samples, warmup=3):
    """Device time per call in ms, `samples` measurements: the calls are captured once into a CUDA graph (host-side
    call overhead stays outside) and every replay is one sample, bracketed by CUDA events on the launching stream."""
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
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(samples + 1)]
    ev[0].record()
    for i in range(samples):
        graph.replay()
        ev[i + 1].record()
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) / len(calls) for i in range(samples)]


def op_specs(sg, seed, bw_rows=None):
    """The other configured ops: name -> (label, flops, compulsory bytes, dtype, make(set) -> buffers, call)."""
    import torch

    def mm(Mx, Nx, Kx, dtype, label):
        es = 2 if dtype == "bf16" else 4
        return (label, 2.0 * Mx * Nx * Kx, (Mx * Kx + Kx * Nx) * es + Mx * Nx * 4, dtype,
                lambda s: (gpu_operand((Mx, Kx), seed, 10 + s, "uniform", dtype),
                           gpu_operand((Kx, Nx), seed, 40 + s, "uniform", dtype), torch.empty(Mx, Nx, device="cuda")),
                lambda a, b, c: sg.sg_matmul(a, b, c))

    def mm_t(Mx, Nx, Kx, a_t, b_t, label, dtype="bf16"):
        # operands stored transposed and handed over as strided views (Section 4.6.1: A^T B, A B^T)
        es = 2 if dtype == "bf16" else 4
        return (label, 2.0 * Mx * Nx * Kx, (Mx * Kx + Kx * Nx) * es + Mx * Nx * 4, dtype,
                lambda s: ((gpu_operand((Kx, Mx), seed, 10 + s, "uniform", dtype).t() if a_t else gpu_operand((Mx, Kx), seed, 10 + s, "uniform", dtype)),
                           (gpu_operand((Nx, Kx), seed, 40 + s, "uniform", dtype).t() if b_t else gpu_operand((Kx, Nx), seed, 40 + s, "uniform", dtype)),
                           torch.empty(Mx, Nx, device="cuda")),
                lambda a, b, c: sg.sg_matmul(a, b, c))

    def dw(Nx, Ho, Wo, Cx, KH, KW, st, dtype, label):
        # bytes by the paper's model (Section 4.6.3): output + filter + input / prod gcd(stride, dilation)
        es = 2 if dtype == "bf16" else 4
        Hi, Wi = (Ho - 1) * st + KH, (Wo - 1) * st + KW
        return (label, 2.0 * Nx * Ho * Wo * Cx * KH * KW, Nx * Ho * Wo * Cx * 4 + KH * KW * Cx * es + Nx * Hi * Wi * Cx * es, dtype,
                lambda s: (gpu_operand((Nx, Hi, Wi, Cx), seed, 130 + s, "normal", dtype), gpu_operand((KH, KW, Cx), seed, 150, "normal", dtype),
                           torch.empty(Nx, Ho, Wo, Cx, device="cuda")),
                lambda i, k, o: sg.sg_depthwise_conv2d_nhwc_hwc(i, k, o, (st, st), (1, 1)))

    bw_cache = {}

    def bw_source(dtype):
        # one seeded tensor per dtype, several times the size of L2; rotating sets are device copies
        if dtype not in bw_cache:
            bw_cache[dtype] = gpu_operand((bw_rows or BW_ROWS, BW_COLS), seed, 170, "uniform", dtype)
        return bw_cache[dtype]

    def bw(kind, dtype, shape=None):
        # the memory-bound 2-D kernels (Section 4.4); bytes = every input element read once, every output written once.
        # shape None: the large tensor above; else a small seeded tensor of its own (the paper's cache-resident sizes)
        es = 2 if dtype == "bf16" else 4
        R, C = shape or (bw_rows or BW_ROWS, BW_COLS)
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        src = (lambda s: gpu_operand((R, C), seed, 171 + s, "uniform", dtype)) if shape else (lambda s: bw_source(dtype).clone())
        if kind == "copy2d":
            return (f"Copy2D {R}x{C} {dtype}", 0.0, 2 * R * C * es, dtype,
                    lambda s: (src(s), torch.empty(R, C, device="cuda", dtype=tdt)), lambda a, o: sg.sg_copy2d(a, o))
        if kind == "transpose2d":
            return (f"Transpose2D {R}x{C} {dtype}", 0.0, 2 * R * C * es, dtype,
                    lambda s: (src(s), torch.empty(C, R, device="cuda", dtype=tdt)), lambda a, o: sg.sg_transpose2d(a, o))
        n_out = C if kind == "colred2d" else R
        fn = sg.sg_colred2d if kind == "colred2d" else sg.sg_rowred2d
        return (f"{'ColRed2D' if kind == 'colred2d' else 'RowRed2D'} {R}x{C} {dtype}", float(R * C), R * C * es + n_out * 4, dtype,
                lambda s: (src(s), torch.empty(n_out, device="cuda")), lambda a, o: fn(a, o))

    def mm_fused(Mx, Nx, Kx, dtype, label):
        # matmul with the pointwise consumer relu(. + bias[n]) folded into its write-back (Sections 2.1, 3.3)
        es = 2 if dtype == "bf16" else 4
        return (label, 2.0 * Mx * Nx * Kx, (Mx * Kx + Kx * Nx) * es + Nx * 4 + Mx * Nx * 4, dtype,
                lambda s: (gpu_operand((Mx, Kx), seed, 10 + s, "uniform", dtype), gpu_operand((Kx, Nx), seed, 40 + s, "uniform", dtype),
                           gpu_operand((Nx,), seed, 60, "normal", "f32"), torch.empty(Mx, Nx, device="cuda")),
                lambda a, b, bias, c: sg.sg_matmul_bias_act(a, b, bias, c, sg.SG_ACT_RELU))

    paper_shape = (250, 960)      # the one size the paper names for these kernels (caption of its L3 bandwidth figure)
    return {
        "copy2d_f32": bw("copy2d", "f32"), "copy2d_bf16": bw("copy2d", "bf16"),
        "transpose2d_f32": bw("transpose2d", "f32"), "transpose2d_bf16": bw("transpose2d", "bf16"),
        "colred2d_f32": bw("colred2d", "f32"), "rowred2d_f32": bw("rowred2d", "f32"),
        "colred2d_bf16": bw("colred2d", "bf16"), "rowred2d_bf16": bw("rowred2d", "bf16"),
        "copy2d_250x960_f32": bw("copy2d", "f32", paper_shape), "transpose2d_250x960_f32": bw("transpose2d", "f32", paper_shape),
        "colred2d_250x960_f32": bw("colred2d", "f32", paper_shape), "rowred2d_250x960_f32": bw("rowred2d", "f32", paper_shape),
        "depthwise_112_f32": dw(1, 112, 112, 32, 3, 3, 1, "f32", "depthwise conv2d 1x114x114x32 * 3x3x32 f32 (MobileNet-like, batch 1)"),
        "depthwise_batched_f32": dw(32, 112, 112, 64, 3, 3, 1, "f32", "depthwise conv2d 32x114x114x64 * 3x3x64 f32"),
        "depthwise_batched_bf16": dw(32, 112, 112, 64, 3, 3, 1, "bf16", "depthwise conv2d 32x114x114x64 * 3x3x64 bf16"),
        "depthwise_batched_s2_f32": dw(32, 56, 56, 128, 3, 3, 2, "f32", "depthwise conv2d 32x113x113x128 * 3x3x128 stride 2 f32"),
        "matmul128_f32": mm(128, 128, 128, "f32", "matmul 128^3 f32 (config 1)"),
        "matmul4096_bf16_atb": mm_t(4096, 4096, 4096, True, False, "matmul 4096^3 bf16, A stored transposed (A^T B)"),
        "matmul4096_bf16_abt": mm_t(4096, 4096, 4096, False, True, "matmul 4096^3 bf16, B stored transposed (A B^T)"),
        "matmul4096_f32_atb": mm_t(4096, 4096, 4096, True, False, "matmul 4096^3 f32, A stored transposed (A^T B)", "f32"),
        "matmul4096_f32_abt": mm_t(4096, 4096, 4096, False, True, "matmul 4096^3 f32, B stored transposed (A B^T)", "f32"),
        "matmul4096_f32": mm(4096, 4096, 4096, "f32", "matmul 4096^3 f32 (sweep corner)"),
        "matmul4096_bf16": mm(4096, 4096, 4096, "bf16", "matmul 4096^3 bf16 (sweep corner)"),
        "matmul1024_bf16": mm(1024, 1024, 1024, "bf16", "matmul 1024^3 bf16 (sweep point)"),
        # a sweep shape of about the step's average size per f32 launch: the shape the DRAM-traffic capture is taken on
        "matmul_2048x2048x1024_f32": mm(2048, 2048, 1024, "f32", "matmul 2048x2048x1024 f32 (sweep point)"),
        "matmul_bias_relu_bf16": mm_fused(4096, 4096, 1024, "bf16", "matmul 4096x4096x1024 bf16 + bias + relu, fused write-back"),
        "matmul4096x4096x1024_bf16": mm(4096, 4096, 1024, "bf16", "matmul 4096x4096x1024 bf16 (the same product, unfused)"),
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


def measure_op(sg, peaks, spec, samples=SAMPLES):
    """Times one op, `samples` measurements.  Cold regime (the one the roofline fraction is quoted from): buffers rotate
    over enough sets to exceed L2 between reuses.  Warm regime, for ops whose operands fit in L2: the same buffers
    every call (the paper's "steady state")."""
    import torch
    label, flops, bytes_, dtype, make, call = spec
    ffma_peak = 148 * 128 * 2 * 1.965e9 / 1e12      # TFLOP/s at the maximum SM clock
    sets = min(16, max(2, int(400e6 // max(bytes_, 1)) + 1))
    bufs = [make(s) for s in range(sets)]
    ncalls = sets * 2 if bytes_ < 100e6 else sets
    calls = [(lambda b=bufs[i % sets]: call(*b)) for i in range(ncalls)]
    call(*bufs[0])
    torch.cuda.synchronize()
    fam, name = sg.sg_last_kernel(), sg.sg_last_kernel_name()
    est_ms = max(flops / 3e14, 5e-3) * ncalls
    samples = int(max(5, min(samples, 2000.0 / est_ms)))        # at most ~2 s of device time per op
    q = quartiles(time_graph(calls, samples))
    ms = q["median"]
    warm = None
    if bytes_ < 100e6:
        warm = quartiles(time_graph([(lambda b=bufs[0]: call(*b)) for _ in range(ncalls)], min(samples, 30)))
    host_ms = time_launches(lambda i: call(*bufs[i % sets]), max(3, min(100, ncalls * 2)), 2)
    tf = flops / (ms * 1e-3) / 1e12
    tensor_peak = peaks["bf16_tflops"] * (TF32_OVER_BF16 if dtype == "f32" else 1.0)
    nominal_peak = NOMINAL_BF16_TFLOPS * (TF32_OVER_BF16 if dtype == "f32" else 1.0)
    on_tensor = fam in (sg.SG_KERNEL_TENSOR, sg.SG_KERNEL_CONV_STRIP)
    t_compute = flops / ((tensor_peak if on_tensor else ffma_peak) * 1e12)
    t_bytes = bytes_ / (peaks["hbm_gbs"] * 1e9)
    bound = max(t_compute, t_bytes)
    row = {"op": label, "dtype": dtype, "kernel": name,
           "us": round(ms * 1e3, 2), "us_p25": round(q["p25"] * 1e3, 2), "us_p75": round(q["p75"] * 1e3, 2),
           "us_mean": round(q["mean"] * 1e3, 2), "samples": q["n"],
           "us_with_host_call": round(host_ms * 1e3, 2), "gflops": round(tf * 1e3, 1),
           "gbs": round(bytes_ / (ms * 1e-3) / 1e9, 1),
           "bound": "hbm" if t_bytes > t_compute else ("tensor" if on_tensor else "ffma"),
           "roofline_us": round(bound * 1e6, 2), "frac": round(bound / (ms * 1e-3), 4), "rotating_sets": sets,
           "timing": "CUDA graph replay, one sample per replay, cold (rotating buffers > L2)"}
    if warm is not None:
        row["us_warm_l2"] = round(warm["median"] * 1e3, 2)
    if on_tensor:
        # against the chip's nominal dense tensor rate (bf16 2250 TFLOP/s, tf32 half of it)
        row["frac_of_nominal_tensor_peak"] = round(tf / nominal_peak, 4)
    if dtype == "f32" and on_tensor:
        # the f32 path issues three tf32 products per term; relative to a third of the MEASURED tf32-equivalent rate
        # (a cuBLAS-derived figure, not a limit of the chip: this ratio can exceed 1)
        row["frac_x3_products_vs_measured"] = round(max(3 * t_compute, t_bytes) / (ms * 1e-3), 4)
    del bufs, calls
    torch.cuda.empty_cache()
    return row


def per_op_table(sg, peaks, seed):
    specs = op_specs(sg, seed)
    return [measure_op(sg, peaks, specs[name]) for name in specs]


def cpu_baseline(target_seconds=12.0, extras=True):
    """Times the oracle, as it stands, on bounded samples of the workloads on the host cores: leading rows of the
    sweep's 4096^3 point with every thread (the contract's `value`) and with one thread, and configs 1, 3 and 4 with
    one thread and with every thread (the paper's own numbers are single-threaded)."""
    import numpy as np
    from oracle import ref
    from paper_2202_03293_b200 import inputs
    seed = inputs.BASE_SEED + 1
    _, b = inputs.make((K, N), seed, 2, "uniform", "bf16")
    threads = ref.max_threads()

    def mm_rows(rows, nthreads):
        _, a = inputs.make((rows, K), seed, 1, "uniform", "bf16")
        t0 = time.perf_counter()
        ref.matmul(a, b, threads=nthreads)
        return time.perf_counter() - t0

    dt = mm_rows(threads, threads)
    rows_full = int(min(M, max(threads, threads * target_seconds / max(dt, 1e-6))))
    rows_full = max(rows_full - rows_full % threads, threads)
    dt = mm_rows(rows_full, threads)
    gflops = 2.0 * rows_full * N * K / dt / 1e9
    info = {"value": round(gflops, 3), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {rows_full} of {M} rows of the 4096^3 matmul ({dt:.1f} s)"}
    if extras:
        others = []
        rows1 = max(1, int(rows_full / threads / 4))
        d1 = mm_rows(rows1, 1)
        others.append({"op": "matmul 4096^3 (sweep corner)", "threads": 1, "gflops": round(2.0 * rows1 * N * K / d1 / 1e9, 3),
                       "sample": f"first {rows1} rows ({d1:.1f} s)"})
        a1, b1 = inputs.uniform((128, 128), seed, 3), inputs.uniform((128, 128), seed, 4)
        i3, k3 = inputs.uniform((16, 1026, 64), seed, 5), inputs.uniform((3, 64, 128), seed, 6)
        i4 = inputs.make((4, 58, 58, 64), seed, 7, "normal", "bf16")[1]
        k4 = inputs.make((3, 3, 64, 128), seed, 8, "normal", "bf16")[1]
        cases = [("matmul 128^3 f32 (config 1)", 2.0 * 128 ** 3, "whole problem", lambda t: ref.matmul(a1, b1, threads=t)),
                 ("conv_1d_nwc_wcf config 3", 2.0 * 16 * 1024 * 128 * 3 * 64, "16 of 32 batch entries", lambda t: ref.conv1d_nwc_wcf(i3, k3, threads=t)),
                 ("conv_2d_nhwc_hwcf config 4", 2.0 * 4 * 56 * 56 * 128 * 9 * 64, "4 of 16 images", lambda t: ref.conv2d_nhwc_hwcf(i4, k4, threads=t))]
        for label, flops, sample, fn in cases:
            for t in (1, threads):
                fn(t)                                   # (the first call also builds and loads the library)
                t0 = time.perf_counter()
                fn(t)
                d = time.perf_counter() - t0
                others.append({"op": label, "threads": t, "gflops": round(flops / d / 1e9, 3), "sample": f"{sample} ({d:.2f} s)"})
        info["others"] = others
    return info, dt, rows_full


def run_reference(args, rank):
    """The reference arm: the paper ships no code, so the CPU oracle is timed, as it stands, on the host cores; a step
    is a bounded sample of the same workload (leading rows of the sweep's largest point)."""
    if rank != 0:
        return
    vals, times = [], []
    info = None
    n = max(1, args.warmup + args.steps)
    for i in range(n):
        info, dt, rows = cpu_baseline(target_seconds=max(1.0, min(10.0, 90.0 / n)), extras=False)
        if i >= args.warmup:
            vals.append(info["value"])
            times.append(dt)
    value = statistics.fmean(vals)
    info["value"] = round(value, 3)
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3),
            "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(statistics.fmean(times) * 1e3, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": "each step: leading rows of the sweep's 4096^3 point, bf16-valued inputs; "
                                                       "ms_per_step is the time of that sample, not of the whole sweep"},
            "cpu_baseline": info, "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0,
                                           "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def sweep_buffers(torch, seed):
    """Dense device buffers for every shape of the sweep, both dtypes: sub-blocks of one seeded
    4096 x 4096 sample per operand, copied out so that every matrix is contiguous."""
    import numpy as np
    from paper_2202_03293_b200 import inputs
    full = {}
    for dtype in ("bf16", "f32"):
        for name, tid in (("A", 1), ("B", 2)):
            payload, _ = inputs.make((4096, 4096), seed, tid, "uniform", dtype)
            t = torch.from_numpy(payload.view(np.int16) if dtype == "bf16" else payload).cuda()
            full[dtype, name] = t.view(torch.bfloat16) if dtype == "bf16" else t
    bufs = {}
    for dtype in ("bf16", "f32"):
        for (m, n, k) in SHAPES:
            bufs[dtype, m, n, k] = (full[dtype, "A"][:m, :k].contiguous(), full[dtype, "B"][:k, :n].contiguous(),
                                    torch.empty(m, n, device="cuda"))
    return bufs


def sweep_table(sg, peaks, bufs, torch):
    """Per-shape device time (CUDA events around a few back-to-back launches) and roofline fraction."""
    rows = []
    for dtype in ("bf16", "f32"):
        es = 2 if dtype == "bf16" else 4
        peak = peaks["bf16_tflops"] * (TF32_OVER_BF16 if dtype == "f32" else 1.0) * 1e12
        for (m, n, k) in SHAPES:
            a, b, c = bufs[dtype, m, n, k]
            flops = 2.0 * m * n * k
            # device time by graph replay of a few back-to-back calls (the host's call overhead stays outside)
            ncalls = int(max(2, min(16, 1e-3 / max(flops / 3e14, 8e-6))))
            ms = statistics.median(time_graph([lambda: sg.sg_matmul(a, b, c)] * ncalls, 5))
            t_c, t_b = flops / peak, ((m * k + k * n) * es + m * n * 4) / (peaks["hbm_gbs"] * 1e9)
            rows.append({"dtype": dtype, "M": m, "N": n, "K": k, "us": round(ms * 1e3, 2),
                         "gflops": round(flops / (ms * 1e-3) / 1e9, 1), "bound": "hbm" if t_b > t_c else "tensor",
                         "frac": round(max(t_c, t_b) / (ms * 1e-3), 4)})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-per-op", action="store_true", help="skip the per-op table")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--streams", type=int, default=4, help="parallel branches of the step's CUDA graphs")
    ap.add_argument("--op", default=None, help="time only this op of the per-op table (used for profiler captures)")
    ap.add_argument("--bw-rows", type=int, default=None,
                    help="with --op: rows of the memory-bound 2-D kernels' tensor (a smaller case for profiler captures)")
    ap.add_argument("--sweep-table", default=None, help="also time every shape of the sweep on its own and write the table to this JSON file")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: start one rank per GPU ourselves (as many as the node has, at most --gpus)
        ranks = min(args.gpus, torch.cuda.device_count())
        if ranks > 1:
            import socket
            with socket.socket() as sock:
                sock.bind(("127.0.0.1", 0))
                port = sock.getsockname()[1]
            argv = [a for a in sys.argv[1:]]
            for i, a in enumerate(argv):            # the ranks are told how many of them there are
                if a == "--gpus":
                    argv[i + 1] = str(ranks)
                elif a.startswith("--gpus="):
                    argv[i] = f"--gpus={ranks}"
            cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={ranks}",
                   "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
            raise SystemExit(subprocess.call(cmd))
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
        specs = op_specs(sg, seed, args.bw_rows)
        if args.op not in specs:
            raise SystemExit(f"--op must be one of {sorted(specs)}")
        if args.steps == 0:
            # a handful of plain launches over two buffer sets and nothing else: the command a profiler capture wraps
            label, flops, bytes_, dtype, make, call = specs[args.op]
            bufs = [make(s) for s in range(2)]
            for i in range(4):
                call(*bufs[i % 2])
            torch.cuda.synchronize()
            sg.sg_check()
            print(json.dumps({"op": label, "kernel": sg.sg_last_kernel_name(), "launched": 4}), flush=True)
            return
        print(json.dumps(measure_op(sg, peaks, specs[args.op], samples=max(1, min(args.steps, SAMPLES)))), flush=True)
        return

    bufs = sweep_buffers(torch, seed)
    # large shapes first, so that the host's call overhead of the small ones hides behind them
    order = sorted(SHAPES, key=lambda s: -s[0] * s[1] * s[2])
    halves = {dt: [bufs[dt, m, n, k] for (m, n, k) in order] for dt in ("f32", "bf16")}
    mid = torch.cuda.Event(enable_timing=True)

    def step(mark=None):
        for a, b, c in halves["f32"]:
            sg.sg_matmul(a, b, c)
        if mark is not None:
            mark.record()
        for a, b, c in halves["bf16"]:
            sg.sg_matmul(a, b, c)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # The 250 calls of a step are captured once into two CUDA graphs (the f32 half and the bf16
    # half) and a step replays them: the launch mechanism a fixed sweep would use in production.
    # The same step issued call by call is timed as well ("eager_ms_per_step").
    for i in range(2):
        step()
    barrier()
    side = torch.cuda.Stream()
    graphs = {}
    launches_per_step = 0
    lanes = [torch.cuda.Stream() for _ in range(max(1, args.streams) - 1)]
    for dt in ("f32", "bf16"):
        g = torch.cuda.CUDAGraph()
        n0 = sg.sg_launch_count()
        with torch.cuda.graph(g, stream=side):
            # the calls are independent (every shape has its own buffers): dealt round-robin onto
            # parallel branches of the graph, small problems overlap and one kernel's last,
            # partly filled wave of tiles runs beside the next kernel's first
            for ln in lanes:
                ln.wait_stream(side)
            for i, (a, b, c) in enumerate(halves[dt]):
                j = i % (len(lanes) + 1)
                if j == 0:
                    sg.sg_matmul(a, b, c)
                else:
                    with torch.cuda.stream(lanes[j - 1]):
                        sg.sg_matmul(a, b, c)
            for ln in lanes:
                side.wait_stream(ln)
        launches_per_step += sg.sg_launch_count() - n0
        graphs[dt] = g

    def graph_step(mark=None):
        graphs["f32"].replay()
        if mark is not None:
            mark.record()
        graphs["bf16"].replay()

    for i in range(warmup):
        graph_step()
    barrier()
    # a few steps split at the dtype boundary: which kernel dominates, and its average launch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f32_ms = bf16_ms = 0.0
    for i in range(3):
        e0.record(); graph_step(mid); e1.record()
        torch.cuda.synchronize()
        f32_ms += e0.elapsed_time(mid); bf16_ms += mid.elapsed_time(e1)

    sampler = ClockSampler(local_rank)
    sampler.start()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    marks[0].record()
    for i in range(args.steps):
        graph_step()
        marks[i + 1].record()
    barrier()
    launches = launches_per_step * args.steps
    clocks = sampler.stop()
    sg.sg_check()
    ms_total = sharding.max_over_ranks(marks[0].elapsed_time(marks[-1]), device="cuda")
    ms_per_step = ms_total / args.steps
    step_q = quartiles([marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)])      # this rank's steps
    value = world * FLOPS_PER_STEP / (ms_per_step * 1e-3) / 1e9      # GFLOP/s, all ranks

    eager_steps = max(3, min(20, args.steps))
    e0.record()
    for i in range(eager_steps):
        step()
    e1.record()
    barrier()
    eager_ms = sharding.max_over_ranks(e0.elapsed_time(e1), device="cuda") / eager_steps

    # ---- end to end through the public call, host buffers, copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        host = {key: (a.cpu().pin_memory(), b.cpu().pin_memory(), torch.empty(c.shape).pin_memory())
                for key, (a, b, c) in bufs.items()}
        e2e_steps = max(2, min(5, args.steps))
        h2d = sum(a.numel() * a.element_size() + b.numel() * b.element_size() for a, b, _ in host.values())
        d2h = sum(c.numel() * 4 for _, _, c in host.values())

        # The calls of a step are independent, so the user-side pipeline is three streams: inputs go up on one,
        # sg_matmul runs on the current one, results come down on a third; events order each shape's copy-in ->
        # matmul -> copy-out, and the next step's reuse of the same device buffers.
        cur = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = {key: torch.cuda.Event() for key in bufs}
        ev_mm = {key: torch.cuda.Event() for key in bufs}
        ev_out = {key: torch.cuda.Event() for key in bufs}
        e2e_order = [(dt, m, n, k) for dt in ("f32", "bf16") for (m, n, k) in order]

        def e2e_step():
            for key in e2e_order:
                a, b, c = bufs[key]
                ah, bh, ch = host[key]
                with torch.cuda.stream(s_in):
                    s_in.wait_event(ev_mm[key])          # the previous step's matmul has read a and b
                    a.copy_(ah, non_blocking=True)
                    b.copy_(bh, non_blocking=True)
                    ev_in[key].record(s_in)
                cur.wait_event(ev_in[key])
                cur.wait_event(ev_out[key])              # the previous step's copy-out has read c
                sg.sg_matmul(a, b, c)
                ev_mm[key].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_mm[key])
                    ch.copy_(c, non_blocking=True)
                    ev_out[key].record(s_out)
            cur.wait_stream(s_in)
            cur.wait_stream(s_out)                       # the step ends when its last result is on the host

        e2e_step()
        barrier()
        e0.record()
        for i in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = sharding.max_over_ranks(e0.elapsed_time(e1), device="cuda")
        e2e = {"value": round(world * FLOPS_PER_STEP / (e2e_ms / e2e_steps * 1e-3) / 1e9, 1), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
        del host

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # dominant kernel: the f32 tensor-core kernel (three tf32 products per term).  Its launches in a
    # step are the 125 f32 shapes; achieved = their algorithmic flops over their device time.
    timed_seconds = ms_total * 1e-3
    peak_kind = "bf16_tflops_sustained" if timed_seconds >= 1.0 else "bf16_tflops"
    tf32_peak = peaks[peak_kind] * TF32_OVER_BF16
    share_f32 = f32_ms / (f32_ms + bf16_ms)
    f32_tf = FLOPS_PER_DTYPE / (ms_per_step * share_f32 * 1e-3) / 1e12
    bf16_tf = FLOPS_PER_DTYPE / (ms_per_step * (1 - share_f32) * 1e-3) / 1e12
    avg_alg_bytes = sum((m * k + k * n) * 4 + m * n * 4 for m, n, k in SHAPES) / len(SHAPES)
    traffic, traffic_note = traffic_per_launch(avg_alg_bytes)
    roofline = {"bound": "tensor", "achieved": round(f32_tf, 1), "peak": round(tf32_peak, 1), "unit": "TFLOP/s",
                "frac": round(f32_tf / tf32_peak, 4), "traffic": traffic, "traffic_source": traffic_note,
                "algorithmic_bytes_per_launch": round(avg_alg_bytes),
                "kernel": "tc_gemm_kernel<BN, CG, f32> (125 launches per step, %.0f%% of the step)" % (100 * share_f32),
                "peak_source": f"{peaks['source']} {peak_kind} x {TF32_OVER_BF16} (tf32 : bf16 tensor rate); timed region {timed_seconds:.2f} s",
                "algorithmic_flops_per_step": FLOPS_PER_DTYPE, "avg_launch_us": round(ms_per_step * share_f32 * 1e3 / len(SHAPES), 2),
                "note": "f32 accuracy costs three tf32 products per term: a third of the tf32 rate is what this kernel can reach; the peak is a measured cuBLAS rate, not a limit of the chip",
                "frac_x3_products_vs_measured": round(3 * f32_tf / tf32_peak, 4),
                "frac_of_nominal_tensor_peak": round(f32_tf / (NOMINAL_BF16_TFLOPS * TF32_OVER_BF16), 4),
                "bf16_half": {"achieved": round(bf16_tf, 1), "peak": peaks[peak_kind], "frac": round(bf16_tf / peaks[peak_kind], 4),
                              "frac_of_nominal_tensor_peak": round(bf16_tf / NOMINAL_BF16_TFLOPS, 4),
                              "share_of_step": round(1 - share_f32, 4)}}

    line = {"metric": METRIC, "value": round(value, 1),
            "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": round(ms_per_step, 5),
            "ms_per_step_samples": {k: (round(v, 5) if k != "n" else v) for k, v in step_q.items()},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16+f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "calls_per_step": 2 * len(SHAPES),
                       "launch": f"each step replays two CUDA graphs holding the step's 250 library calls on {max(1, args.streams)} parallel branches",
                       "l2": "every shape has its own buffers, 6.3 GB per step > 126 MB L2",
                       "parallelism": f"replicas x{world}, no collective"},
            "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches),
            "eager_ms_per_step": round(eager_ms, 5), "e2e": e2e}
    if args.sweep_table:
        rows = sweep_table(sg, peaks, bufs, torch)
        with open(args.sweep_table, "w") as f:
            json.dump(rows, f)
        for dt in ("bf16", "f32"):
            fr = sorted(r["frac"] for r in rows if r["dtype"] == dt)
            line.setdefault("sweep_fractions", {})[dt] = {"min": fr[0], "median": fr[len(fr) // 2], "max": fr[-1]}
    del bufs, halves
    torch.cuda.empty_cache()
    if not args.no_per_op:
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
