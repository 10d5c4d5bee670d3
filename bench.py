#!/usr/bin/env python
"""Benchmark of the MX hot path on B200: quantize / dequantize GB/s and block-scaled
GEMM TFLOP/s on seeded synthetic tensors shaped like the paper's transformer
workloads (arXiv 2310.10537).

One step = one pass of the whole hot path:
  sweep   the 8192 x 8192 BF16 tensor of the quantize/dequantize sweep, cast to each of
          the six MX formats (blocks along the last axis, scales in the layout the
          GEMM reads) and dequantized back to BF16                      [12 launches]
  ffn     the FFN up-projection: quantize X[8192 x 4096] along its contiguous axis,
          W[4096 x 16384] along its strided axis (transposing requantize), then the
          MXFP8 block-scaled GEMM 8192 x 16384 x 4096 with FP32 output  [3 launches]
`value` is the algorithmic GB/s of the sweep (the configuration the quantize metric is
quoted on); the GEMM and the other phases are reported beside it in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
Under torchrun every rank runs the same step on its own GPU (weak scaling, no
exchange: MX blocks are independent) and rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FMT_NAMES = ["e4m3", "e5m2", "e3m2", "e2m3", "e2m1", "int8"]
FMT_BITS = [8, 8, 6, 6, 4, 8]
SWEEP_ROWS, SWEEP_COLS = 8192, 8192
FFN_TOKENS, FFN_IN, FFN_OUT = 8192, 4096, 16384


def algorithmic_bytes(numel: int, in_bytes: int, bits: int) -> float:
    """Bytes a quantize (or dequantize) pass must move: float tensor + codes + one scale per 32."""
    return numel * (in_bytes + bits / 8.0 + 1.0 / 32.0)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def max_over_ranks(values, device, world: int):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the job's
    time).  With one rank it is the identity; otherwise an all-reduce on the process group that
    is already initialised (NCCL on GPUs, gloo in the CPU tests)."""
    import torch
    if world <= 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(units_per_rank: float, world: int, slowest_seconds: float) -> float:
    """Whole-job throughput under weak scaling: every rank processes `units_per_rank` of its own
    shard (MX blocks are independent, so ranks exchange nothing) in the time of the slowest rank."""
    return world * units_per_rank / slowest_seconds


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU with nvidia-smi (a process of its
    own, started well before the timed region so that it is already polling) while the timed region
    runs.  Every sample carries nvidia-smi's timestamp; the caller marks the timed region with
    begin() / end(), both right after a device synchronize, and the samples inside that window are
    the ones reported.  If the window caught none (a very short run), the samples taken under load
    -- power above half of the maximum seen -- stand in, and the result says so."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.proc = None
        self.t0 = self.t1 = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "10"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    @staticmethod
    def _epoch(stamp: str):
        import datetime
        try:
            return datetime.datetime.strptime(stamp, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        return self.summarize(out, self.t0, self.t1)

    @classmethod
    def summarize(cls, text: str, t0, t1):
        """The clocks record from nvidia-smi's CSV lines and the timed region's host times."""
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        samples = []  # (epoch or None, sm, max sm, power, reasons)
        for line in text.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm, mx_, power = float(parts[1]), float(parts[2]), float(parts[3])
            except ValueError:
                continue
            samples.append((cls._epoch(parts[0]), sm, mx_, power,
                            {n for n, v in zip(names, parts[4:8]) if v.lower().startswith("active")}))
        if not samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        inside = [x for x in samples if x[0] is not None and t0 is not None and t0 <= x[0] <= t1]
        pmax = max(x[3] for x in samples)
        use = inside or [x for x in samples if x[3] > 0.5 * pmax] or samples
        return {"sm_mhz": statistics.median(x[1] for x in use), "sm_max_mhz": max(x[2] for x in samples),
                "samples": len(use), "in_timed_region": bool(inside),
                "power_w_median": statistics.median(x[3] for x in use),
                "power_w_max": max(x[3] for x in use), "reasons": sorted(set().union(*[x[4] for x in use]))}


# --------------------------------------------------------------------------------------
# our arm: the CUDA library through its Python binding
# --------------------------------------------------------------------------------------

class Workload:
    def __init__(self, torch, mx, inputs, device, seed_offset: int):
        self.torch, self.mx = torch, mx
        T = inputs.config2(device, SWEEP_ROWS, SWEEP_COLS, seed=2002 + seed_offset)
        self.T = [T, T.clone()]  # two copies, read alternately: no launch re-reads what L2 still holds
        shape = [SWEEP_ROWS, SWEEP_COLS]
        u8 = dict(dtype=torch.uint8, device=device)
        self.sweep = []
        for fmt in range(6):
            e = torch.empty(mx.mx_elems_bytes(shape, 1, fmt), **u8)
            s = torch.empty(mx.mx_scales_bytes(shape, 1), **u8)
            d = torch.empty(shape, dtype=torch.bfloat16, device=device)
            self.sweep.append((e, s, d))
        f = inputs.config3(device, FFN_TOKENS, FFN_IN, FFN_OUT, seed=3003 + seed_offset)
        self.X, self.W = f["X"], f["W"]
        self.ea = torch.empty(mx.mx_elems_bytes([FFN_TOKENS, FFN_IN], 1, mx.MX_E4M3), **u8)
        self.sa = torch.empty(mx.mx_scales_bytes([FFN_TOKENS, FFN_IN], 1), **u8)
        self.eb = torch.empty(mx.mx_elems_bytes([FFN_IN, FFN_OUT], 0, mx.MX_E4M3), **u8)
        self.sb = torch.empty(mx.mx_scales_bytes([FFN_IN, FFN_OUT], 0), **u8)
        self.C = torch.empty((FFN_TOKENS, FFN_OUT), dtype=torch.float32, device=device)
        # L2 flush: a READ of 512 MB (four times the 126 MB L2).  Reading evicts what the kernel
        # before left behind -- its dirty lines are written back while the flush runs, not while
        # the next phase is being timed -- and leaves the cache full of clean, unrelated lines.
        self.flush_buf = torch.zeros(128 << 20, dtype=torch.int32, device=device)
        self.flush_out = torch.zeros((), dtype=torch.int32, device=device)
        n = SWEEP_ROWS * SWEEP_COLS
        self.bytes_q = [algorithmic_bytes(n, 2, b) for b in FMT_BITS]
        self.bytes_sweep = 2.0 * sum(self.bytes_q)
        self.bytes_qx = algorithmic_bytes(FFN_TOKENS * FFN_IN, 2, 8)
        self.bytes_qw = algorithmic_bytes(FFN_IN * FFN_OUT, 2, 8)
        self.flops = 2.0 * FFN_TOKENS * FFN_OUT * FFN_IN
        self.launches_per_step = 15

    def flush_l2(self):
        self.torch.amax(self.flush_buf, dim=0, out=self.flush_out)

    N_EVENTS = 9

    def step(self, ev=None):
        """One pass of the hot path.  ev: list of N_EVENTS CUDA events bracketing the phases; every
        phase starts behind an L2 flush that lies outside its own timer."""
        torch, mx = self.torch, self.mx
        rec = (lambda i: ev[i].record()) if ev is not None else (lambda i: None)
        self.flush_l2()      # the step starts cold too (before it: the GEMM's 537 MB of output)
        rec(0)
        for fmt in range(6):                                   # a1-a4: float -> MX, last axis
            e, s, _ = self.sweep[fmt]
            mx.mx_quantize(self.T[fmt & 1], 1, fmt, mx.MX_RNE, mx.MX_SCALES_SWIZZLED, out=(e, s))
        rec(1)
        for fmt in range(6):                                   # a6: MX -> BF16
            e, s, d = self.sweep[fmt]
            mx.mx_dequantize(e, s, [SWEEP_ROWS, SWEEP_COLS], fmt, torch.bfloat16,
                             mx.MX_SCALES_SWIZZLED, out=d)
        rec(2)
        self.flush_l2()
        rec(3)
        mx.mx_quantize(self.X, 1, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED, out=(self.ea, self.sa))
        rec(4)
        self.flush_l2()
        rec(5)
        mx.mx_quantize(self.W, 0, mx.MX_E4M3, mx.MX_RNE, mx.MX_SCALES_SWIZZLED, out=(self.eb, self.sb))  # a5
        rec(6)
        self.flush_l2()
        rec(7)
        mx.mx_gemm(self.ea, self.sa, self.eb, self.sb, FFN_TOKENS, FFN_OUT, FFN_IN,       # a7-a9
                   mx.MX_E4M3, mx.MX_E4M3, out=self.C)
        rec(8)


def run_e2e(torch, mx, inputs, steps: int, warmup: int):
    """The sweep through the host-buffer entry points: pinned host tensors in, pinned host
    results out, every copy inside the timed region."""
    T = inputs.config2("cpu", SWEEP_ROWS, SWEEP_COLS, seed=2002).pin_memory()  # the whole sweep tensor
    rows, cols = T.shape
    shape = [rows, cols]
    n = rows * cols
    bufs, outs, wss = [], [], []
    for fmt in range(6):
        e = torch.empty(mx.mx_elems_bytes(shape, 1, fmt), dtype=torch.uint8).pin_memory()
        s = torch.empty(mx.mx_scales_bytes(shape, 1), dtype=torch.uint8).pin_memory()
        bufs.append((e, s))
        outs.append(torch.empty(shape, dtype=torch.bfloat16).pin_memory())
        wss.append(torch.empty(mx.mx_quantize_host_workspace_bytes(shape, 1, fmt, torch.bfloat16),
                               dtype=torch.uint8, device="cuda"))
    h2d = d2h = 0

    def one():
        # the six quantizes are queued back to back (the upload of one overlaps the download of the
        # one before), then waited for; the six dequantizes likewise
        nonlocal h2d, d2h
        h2d = d2h = 0
        for fmt in range(6):
            e, s = bufs[fmt]
            mx.mx_quantize_host(T, e, s, 1, fmt, mx.MX_RNE, wss[fmt], queue=True)
            h2d += T.numel() * 2
            d2h += e.numel() + s.numel()
        mx.mx_host_synchronize()
        for fmt in range(6):
            e, s = bufs[fmt]
            mx.mx_dequantize_host(e, s, outs[fmt], fmt, wss[fmt], queue=True)
            h2d += e.numel() + s.numel()
            d2h += outs[fmt].numel() * 2
        mx.mx_host_synchronize()

    for _ in range(max(1, warmup)):
        one()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / steps
    total_bytes = 2.0 * sum(algorithmic_bytes(n, 2, b) for b in FMT_BITS)
    return {"value": total_bytes / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": dt * 1e3,
            "workload": f"configs[1] sweep on the whole {rows}x{cols} BF16 tensor via mx_quantize_host_async / "
                        "mx_dequantize_host_async + mx_host_synchronize (pinned host buffers, copies timed)"}


def run_extras(torch, mx, inputs, peaks, gpu_index):
    """The other benchmark configurations, outside the timed step: the FP4-weight x FP8-activation
    GEMM (16384 x 28672 x 8192), the same shape with both operands FP4 (kind::mxf4), and the
    MXFP6 training step of one 4096^3 linear layer (six quantizes, three GEMMs).  Returns
    (other_configs, gemm_rooflines): the second holds, per configuration, the burst figure against
    2 x the measured BF16 burst peak and -- for configurations 3 and 5 -- a loop of at least two
    seconds of back-to-back launches against 2 x the measured sustained BF16 peak, with the SM
    clock and board power sampled inside that loop."""
    fp8_burst, fp8_sust = 2.0 * peaks["bf16_tflops"], 2.0 * peaks["bf16_tflops_sustained"]
    rooflines = {}

    def burst_entry(flops, seconds):
        tf = flops / seconds / 1e12
        return {"TFLOPs": tf, "ms": seconds * 1e3, "frac_of_2x_bf16_burst": tf / fp8_burst,
                "frac_of_nominal_4500": tf / 4500.0}

    def sustained(fn, flops, t_one, seconds=2.2):
        """fn() queued back to back for >= `seconds`; clocks and power from the samples inside."""
        n = max(4, int(seconds / t_one) + 1)
        sampler = ClockSampler(gpu_index)
        time.sleep(0.3)                      # the sampler is polling before the loop starts
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.begin()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        sampler.end()
        clk = sampler.stop()
        sec = e0.elapsed_time(e1) * 1e-3
        tf = flops * n / sec / 1e12
        return {"TFLOPs": tf, "seconds": sec, "launches": n, "frac_of_2x_bf16_sustained": tf / fp8_sust,
                "frac_of_nominal_4500": tf / 4500.0, "sm_mhz_median": clk.get("sm_mhz"),
                "power_w_median": clk.get("power_w_median"), "power_w_max": clk.get("power_w_max"),
                "clock_samples": clk.get("samples"), "reasons": clk.get("reasons")}

    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    out = {}
    d = inputs.config5("cuda")
    W, X = d["W"], d["X"]
    M, K = X.shape
    N = W.shape[1]
    ea, sa = mx.mx_quantize(X, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(W, 0, mx.MX_E2M1)
    t_qw = timed(lambda: mx.mx_quantize(W, 0, mx.MX_E2M1, out=(eb, sb)), 5)
    t_qx = timed(lambda: mx.mx_quantize(X, 1, mx.MX_E4M3, out=(ea, sa)), 5)
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    t = timed(lambda: mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E2M1, out=C), 5)
    rooflines["config5"] = {"workload": "configs[4] E4M3 x E2M1 16384x28672x8192, FP32 out",
                            "burst": burst_entry(2.0 * M * N * K, t)}
    c5 = (ea, sa, eb, sb, C, M, N, K, t)
    out["config5_mxfp4_weights_x_mxfp8_activations"] = {
        "gemm_TFLOPs": 2.0 * M * N * K / t / 1e12, "gemm_ms": t * 1e3,
        "quantize_w_strided_GBps": algorithmic_bytes(K * N, 2, 4) / t_qw / 1e9,
        "quantize_x_GBps": algorithmic_bytes(M * K, 2, 8) / t_qx / 1e9}
    ea4, sa4 = mx.mx_quantize(X, 1, mx.MX_E2M1)
    t4 = timed(lambda: mx.mx_gemm(ea4, sa4, eb, sb, M, N, K, mx.MX_E2M1, mx.MX_E2M1, out=C), 5)
    out["mxfp4_x_mxfp4_same_shape_kind_mxf4"] = {"gemm_TFLOPs": 2.0 * M * N * K / t4 / 1e12, "gemm_ms": t4 * 1e3}
    del d, W, X, ea4, sa4
    torch.cuda.empty_cache()
    # two chained products (configs[2] shape): the first one's result requantized to MXFP8 for the next
    d = inputs.config3("cuda")
    X, W = d["X"], d["W"]
    M, K = X.shape
    N = W.shape[1]
    ea, sa = mx.mx_quantize(X, 1, mx.MX_E4M3)
    eb, sb = mx.mx_quantize(W, 0, mx.MX_E4M3)
    C = torch.empty((M, N), dtype=torch.float32, device="cuda")
    qe, qs = mx.mx_quantize(C, 1, mx.MX_E4M3)
    t3 = timed(lambda: mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, out=C), 10)
    rooflines["config3"] = {"workload": "configs[2] E4M3 x E4M3 8192x16384x4096, FP32 out",
                            "burst": burst_entry(2.0 * M * N * K, t3)}
    c3 = (ea, sa, eb, sb, C, M, N, K, t3)

    def gemm_then_quantize():
        mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, out=C)
        mx.mx_quantize(C, 1, mx.MX_E4M3, out=(qe, qs))

    t2 = timed(gemm_then_quantize, 10)
    t1 = timed(lambda: mx.mx_gemm_quantize(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, mx.MX_E4M3,
                                           mx.MX_RNE, elems=qe, scales=qs), 10)
    Cb = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    tb = timed(lambda: mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, out=Cb), 10)
    out["config3_gemm_output_variants"] = {
        "ms_gemm_fp32_then_quantize_e4m3": t2 * 1e3, "ms_gemm_with_quantizing_epilogue": t1 * 1e3,
        "quantizing_epilogue_TFLOPs": 2.0 * M * N * K / t1 / 1e12,
        "ms_gemm_bf16_out": tb * 1e3, "bf16_out_TFLOPs": 2.0 * M * N * K / tb / 1e12}
    # Reference point, not part of the path: the vendor library's MXFP8 GEMM (torch._scaled_mm) on the
    # very same packed operands and swizzled scales, timed in alternation with mx_gemm_bf16.
    try:
        a8 = ea.view(torch.float8_e4m3fn).view(M, K)
        b8 = eb.view(torch.float8_e4m3fn).view(N, K)
        s_a, s_b = sa.view(torch.float8_e8m0fnu), sb.view(torch.float8_e8m0fnu)
        ref = torch._scaled_mm(a8, b8.t(), scale_a=s_a, scale_b=s_b, out_dtype=torch.bfloat16)
        mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, out=Cb)
        same = bool(torch.equal(ref, Cb))
        del ref
        t_ours, t_lib = [], []
        for _ in range(4):
            t_ours.append(timed(lambda: mx.mx_gemm_bf16(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, mx.MX_E4M3, out=Cb), 4))
            t_lib.append(timed(lambda: torch._scaled_mm(a8, b8.t(), scale_a=s_a, scale_b=s_b,
                                                        out_dtype=torch.bfloat16), 4))
        out["config3_vendor_library_reference_bf16_out"] = {
            "mx_gemm_bf16_TFLOPs": 2.0 * M * N * K / statistics.median(t_ours) / 1e12,
            "torch_scaled_mm_TFLOPs": 2.0 * M * N * K / statistics.median(t_lib) / 1e12,
            "outputs_bit_identical": same}
        del a8, b8, s_a, s_b
    except Exception as e:  # a torch build without block-scaled _scaled_mm: no reference point
        out["config3_vendor_library_reference_bf16_out"] = {"unavailable": str(e)[:120]}
    # MXINT8 x MXINT8 on the same shape: dequantize to BF16 + dense BF16 tensor-core GEMM
    ea8, sa8 = mx.mx_quantize(X, 1, mx.MX_INT8)
    eb8, sb8 = mx.mx_quantize(W, 0, mx.MX_INT8)
    ws = torch.empty(mx.mx_gemm_dense_workspace_bytes(M, N, K), dtype=torch.uint8, device="cuda")
    t8 = timed(lambda: mx.mx_gemm_dense(ea8, sa8, eb8, sb8, M, N, K, mx.MX_INT8, mx.MX_INT8,
                                        workspace=ws, out=C), 10)
    out["config3_mxint8_x_mxint8_bf16_route"] = {
        "ms_two_dequantizes_and_dense_gemm": t8 * 1e3, "TFLOPs": 2.0 * M * N * K / t8 / 1e12}
    del d, W, X, Cb, qe, qs, ea8, sa8, eb8, sb8, ws
    torch.cuda.empty_cache()
    d = inputs.config4("cuda")
    Xc, Wc, dY = d["X"], d["W"], d["dY"]
    n = Xc.shape[0]
    act, wt, rnd = mx.MX_E3M2, mx.MX_E2M3, mx.MX_RHAZ
    Y = torch.empty((n, n), dtype=torch.float32, device="cuda")

    # every output buffer exists before the timed loops (no allocator calls inside them)
    q = {k: mx.mx_quantize(t, ax, f, rnd) for k, (t, ax, f) in
         {"xa": (Xc, 1, act), "wb": (Wc, 0, wt), "ga": (dY, 1, act), "wb2": (Wc, 1, wt), "xt": (Xc, 0, act),
          "gt": (dY, 0, act)}.items()}

    def train_step():
        mx.mx_quantize(Xc, 1, act, rnd, out=q["xa"])
        mx.mx_quantize(Wc, 0, wt, rnd, out=q["wb"])
        mx.mx_gemm(*q["xa"], *q["wb"], n, n, n, act, wt, out=Y)            # Y = X W
        mx.mx_quantize(dY, 1, act, rnd, out=q["ga"])
        mx.mx_quantize(Wc, 1, wt, rnd, out=q["wb2"])
        mx.mx_gemm(*q["ga"], *q["wb2"], n, n, n, act, wt, out=Y)           # dX = dY W^T
        mx.mx_quantize(Xc, 0, act, rnd, out=q["xt"])
        mx.mx_quantize(dY, 0, act, rnd, out=q["gt"])
        mx.mx_gemm(*q["xt"], *q["gt"], n, n, n, act, act, out=Y)           # dW = X^T dY

    def train_step_fused():  # each tensor is read once: both of its MX tensors come from one pass
        mx.mx_quantize_dual(Xc, act, rnd, out=(q["xa"], q["xt"]))
        mx.mx_quantize_dual(Wc, wt, rnd, out=(q["wb2"], q["wb"]))
        mx.mx_quantize_dual(dY, act, rnd, out=(q["ga"], q["gt"]))
        mx.mx_gemm(*q["xa"], *q["wb"], n, n, n, act, wt, out=Y)
        mx.mx_gemm(*q["ga"], *q["wb2"], n, n, n, act, wt, out=Y)
        mx.mx_gemm(*q["xt"], *q["gt"], n, n, n, act, act, out=Y)

    # the two variants in alternation (what ran before colours a GEMM-heavy timing), medians
    ts_all, tf_all = [], []
    for _ in range(5):
        ts_all.append(timed(train_step, 6))
        tf_all.append(timed(train_step_fused, 6))
    ts, tf = sorted(ts_all)[2], sorted(tf_all)[2]
    out["config4_mxfp6_training_step"] = {
        "ms_six_quantizes_three_gemms": ts * 1e3, "ms_three_dual_quantizes_three_gemms": tf * 1e3,
        "gemm_flops_per_step": 3 * 2.0 * n ** 3}
    # convolution (Section 4.1 counts it among the dot-product operations): N 32, 56 x 56, C 256 -> 256, 3 x 3
    xc = torch.randn((32, 56, 56, 256), device="cuda", dtype=torch.bfloat16)
    wc = torch.randn((256, 3 * 3 * 256), device="cuda", dtype=torch.bfloat16) * 0.05
    geom = mx.mx_conv_geometry(32, 56, 56, 256, 3, 3, (1, 1), (1, 1), (1, 1))
    Mc, Kc = 32 * 56 * 56, 3 * 3 * 256
    exc, sxc = mx.mx_quantize(xc, 3, mx.MX_E4M3)
    ewc, swc = mx.mx_quantize(wc, 1, mx.MX_E4M3)
    eac, sac = mx.mx_im2col(exc, sxc, geom, mx.MX_E4M3)
    yc = torch.empty((Mc, 256), dtype=torch.float32, device="cuda")
    t_q = timed(lambda: mx.mx_quantize(xc, 3, mx.MX_E4M3, out=(exc, sxc)), 20)
    t_i = timed(lambda: mx.mx_im2col(exc, sxc, geom, mx.MX_E4M3), 20)
    t_g = timed(lambda: mx.mx_gemm(eac, sac, ewc, swc, Mc, 256, Kc, mx.MX_E4M3, mx.MX_E4M3, out=yc), 20)
    t_c = timed(lambda: mx.mx_conv2d(exc, sxc, ewc, swc, geom, 256, mx.MX_E4M3, mx.MX_E4M3, out=yc), 20)
    out["conv_n32_56x56_c256_to_256_3x3_e4m3"] = {
        "us_quantize_x": t_q * 1e6, "us_materialized_im2col": t_i * 1e6, "us_gemm_on_materialized_operand": t_g * 1e6,
        "us_conv2d_operand_fetched_in_gemm": t_c * 1e6, "conv2d_TFLOPs": 2.0 * Mc * 256 * Kc / t_c / 1e12}
    del xc, wc, exc, sxc, ewc, swc, eac, sac, yc
    torch.cuda.empty_cache()
    # the three products of the step, each on its own (operands quantized beforehand)
    (xa, xt), (wb2, wb), (ga, gt) = (mx.mx_quantize_dual(Xc, act, rnd), mx.mx_quantize_dual(Wc, wt, rnd),
                                     mx.mx_quantize_dual(dY, act, rnd))
    c4 = {}
    for name, a_, b_, fb_ in (("forward", xa, wb, wt), ("dgrad", ga, wb2, wt), ("wgrad", xt, gt, act)):
        tt = timed(lambda: mx.mx_gemm(*a_, *b_, n, n, n, act, fb_, out=Y), 20)
        c4[name] = burst_entry(2.0 * n ** 3, tt)
    rooflines["config4"] = {"workload": "configs[3] MXFP6 4096^3: forward E3M2 x E2M3, dgrad E3M2 x E2M3, "
                                        "wgrad E3M2 x E3M2, FP32 out", "burst": c4}
    del d, Xc, Wc, dY, Y, xa, xt, wb2, wb, ga, gt
    torch.cuda.empty_cache()
    # last: the two-second loops
    for key, (ea, sa, eb, sb, C, M, N, K, t_one), fb_ in (("config3", c3, mx.MX_E4M3), ("config5", c5, mx.MX_E2M1)):
        time.sleep(1.0)
        rooflines[key]["sustained"] = sustained(
            lambda: mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, fb_, out=C), 2.0 * M * N * K, t_one)
    return out, rooflines


def run_report(torch, mx, inputs):
    """The per-kernel measurement protocol, as markdown on stdout (kept in BENCH.md): every kernel of
    every benchmark configuration, 10 warm-up launches, then 50 launches each timed with its own pair
    of CUDA events (median and best) and the same 50 launches timed as one back-to-back run, rotating
    over buffer sets larger than twice the L2; the GEMMs also as a two-second sustained loop; the
    oracle's GEMM on a slab of configuration 3 on the host cores."""
    import numpy as np

    import oracle as O
    peaks = measured_peaks()
    hbm, hbm_nom = peaks["hbm_gbs"], 8000.0
    fp8_burst, fp8_sust, fp8_nom = 2 * peaks["bf16_tflops"], 2 * peaks["bf16_tflops_sustained"], 4500.0
    lines = []

    def protocol(fn_of_i, n_sets, reps=50, warm=10):
        for i in range(warm):
            fn_of_i(i % n_sets)
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for i, (a, b) in enumerate(ev):
            a.record()
            fn_of_i(i % n_sets)
            b.record()
        torch.cuda.synchronize()
        each = sorted(a.elapsed_time(b) * 1e-3 for a, b in ev)
        runs = []
        for _ in range(2):  # the faster of two back-to-back runs (the first one after a change of kernel can catch the clocks mid-ramp)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(reps):
                fn_of_i(i % n_sets)
            b.record()
            torch.cuda.synchronize()
            runs.append(a.elapsed_time(b) * 1e-3 / reps)
        return each[len(each) // 2], each[0], min(runs)

    def stream_row(name, byts, times):
        med, best, b2b = times
        lines.append(f"| {name} | {byts / 1e6:.1f} | {med * 1e6:.1f} | {best * 1e6:.1f} | {b2b * 1e6:.1f} | "
                     f"{byts / b2b / 1e9:.0f} | {100 * byts / b2b / 1e9 / hbm:.1f} | {100 * byts / b2b / 1e9 / hbm_nom:.1f} |")

    lines += ["## Quantize / dequantize (HBM-bound)", "",
              f"Peaks: measured copy {hbm:.1f} GB/s, nominal {hbm_nom:.0f} GB/s (80 % of nominal = 6400 GB/s = "
              f"{100 * 6400 / hbm:.1f} % of the measured copy peak).  Times in µs: median and best of 50 launches "
              "timed one by one, and the mean of the same 50 launches back to back, the faster of two such runs "
              "(what a stream of conversions sees; the launches overlap their neighbours' tails).", "",
              "| kernel, config | MB | median | best | back-to-back | GB/s | % measured | % nominal |",
              "|---|---|---|---|---|---|---|---|"]

    def quantize_rows(label, X, axis, fmts, rounding=0):
        shape = list(X.shape)
        n, esz = X.numel(), X.element_size()
        Xs = [X, X.clone(), X.clone()]
        for fmt in fmts:
            outs = [mx.mx_quantize(Xs[0], axis, fmt, rounding) for _ in range(3)]
            t = protocol(lambda i: mx.mx_quantize(Xs[i], axis, fmt, rounding, out=outs[i]), 3)
            stream_row(f"quantize {label} -> {FMT_NAMES[fmt]} (axis {axis})", algorithmic_bytes(n, esz, FMT_BITS[fmt]), t)
            if axis == len(shape) - 1:
                ds = [torch.empty_like(X) for _ in range(3)]
                t = protocol(lambda i: mx.mx_dequantize(outs[i][0], outs[i][1], shape, fmt, X.dtype, out=ds[i]), 3)
                stream_row(f"dequantize {FMT_NAMES[fmt]} -> {label}", algorithmic_bytes(n, esz, FMT_BITS[fmt]), t)
                del ds
            del outs
        del Xs
        torch.cuda.empty_cache()

    quantize_rows("C2 BF16 8192x8192", inputs.config2("cuda"), 1, range(6))
    d3 = inputs.config3("cuda")
    quantize_rows("C3 X BF16 8192x4096", d3["X"], 1, [0])
    quantize_rows("C3 W BF16 4096x16384", d3["W"], 0, [0])
    d4 = inputs.config4("cuda")
    quantize_rows("C4 X FP32 4096x4096 (half-away)", d4["X"], 1, [2], 1)
    quantize_rows("C4 X FP32 4096x4096 (half-away)", d4["X"], 0, [2], 1)
    quantize_rows("C4 W FP32 4096x4096 (half-away)", d4["W"], 0, [3], 1)
    d5 = inputs.config5("cuda")
    quantize_rows("C5 X BF16 16384x8192", d5["X"], 1, [0])
    quantize_rows("C5 W BF16 8192x28672", d5["W"], 0, [4])

    def dual_rows(label, X, fmts, rounding=0):
        # both MX tensors of X from one read: in + 2 x (codes + scales) bytes
        n, esz = X.numel(), X.element_size()
        Xs = [X, X.clone(), X.clone()]
        for fmt in fmts:
            outs = [mx.mx_quantize_dual(Xs[0], fmt, rounding) for _ in range(3)]
            t = protocol(lambda i: mx.mx_quantize_dual(Xs[i], fmt, rounding, out=outs[i]), 3)
            stream_row(f"quantize both axes {label} -> {FMT_NAMES[fmt]}",
                       2 * algorithmic_bytes(n, esz, FMT_BITS[fmt]) - n * esz, t)
            del outs
        del Xs
        torch.cuda.empty_cache()

    dual_rows("C2 BF16 8192x8192", inputs.config2("cuda"), [0, 2, 4])
    dual_rows("C4 X FP32 4096x4096 (half-away)", d4["X"], [2], 1)
    dual_rows("C4 W FP32 4096x4096 (half-away)", d4["W"], [3], 1)

    # decode-shaped products: a few rows of activations against a weight matrix (the weights are read once);
    # measured before the tensor-bound loops, which leave the SM clock low for a while
    lines += ["", "## GEMM with few rows of A (HBM-bound on the weights)", "",
              "Bytes = weight codes + weight scales (what has to come from HBM once); columns as in the first table.", "",
              "| shape, formats | MB | median | best | back-to-back | GB/s | % measured | % nominal |",
              "|---|---|---|---|---|---|---|---|"]
    g = torch.Generator(device="cuda").manual_seed(2024)
    for (M, N, K, fb) in ((16, 16384, 4096, 0), (16, 28672, 8192, 0), (64, 28672, 8192, 0), (16, 28672, 8192, 2),
                          (16, 28672, 8192, 4)):
        A = torch.randn((M, K), generator=g, device="cuda", dtype=torch.bfloat16)
        ea, sa = mx.mx_quantize(A, 1, 0)
        Ws = []
        for _ in range(3):
            W = torch.randn((N, K), generator=g, device="cuda", dtype=torch.bfloat16) * 0.02
            Ws.append(mx.mx_quantize(W, 1, fb))
            del W
        C = torch.empty((M, N), dtype=torch.float32, device="cuda")
        t = protocol(lambda i: mx.mx_gemm(ea, sa, Ws[i][0], Ws[i][1], M, N, K, 0, fb, out=C), 3)
        stream_row(f"{M} x {N} x {K}, E4M3 activations x {FMT_NAMES[fb]} weights", Ws[0][0].numel() + Ws[0][1].numel(), t)
        del Ws, C
        torch.cuda.empty_cache()

    lines += ["", "## GEMM (tensor-bound)", "",
              f"Peaks: 2 x measured BF16 burst = {fp8_burst:.0f} TFLOP/s, 2 x measured BF16 sustained = "
              f"{fp8_sust:.0f}, nominal dense FP8 {fp8_nom:.0f}.  Columns as above; `sustained` = a loop of at "
              "least two seconds of back-to-back launches (the clocks sag under the power cap).", "",
              "| config | GFLOP | median µs | best µs | back-to-back µs | TFLOP/s | % 2xBF16 burst | % nominal | sustained TFLOP/s | % 2xBF16 sustained |",
              "|---|---|---|---|---|---|---|---|---|---|"]

    pending = []   # sustained loops run after every burst measurement: two seconds under the power
                   # cap leave the clocks low for a while and would colour the next row

    def gemm_row(label, A, B, axisA, axisB, fa, fb, M, N, K, rounding=0):
        ea, sa = mx.mx_quantize(A, axisA, fa, rounding)
        eb, sb = mx.mx_quantize(B, axisB, fb, rounding)
        Cs = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(2)]
        # warm-up by time (30 ms): the SM clock needs tens of milliseconds of load to
        # come up, which ten launches of a 70 us kernel do not give it
        fn = lambda i: mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=Cs[i])
        fn(0)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        k = 0
        while time.perf_counter() - t0 < 0.03:
            fn(k & 1)
            k += 1
            if k % 64 == 0:
                torch.cuda.synchronize()
        med, best, b2b = protocol(fn, 2, reps=50)
        del Cs
        torch.cuda.empty_cache()
        pending.append((label, (ea, sa, eb, sb), (fa, fb, M, N, K), (med, best, b2b)))
        return ea, sa, eb, sb

    def sustained_rows():
        for label, (ea, sa, eb, sb), (fa, fb, M, N, K), (med, best, b2b) in pending:
            Cs = [torch.empty((M, N), dtype=torch.float32, device="cuda") for _ in range(2)]
            flops = 2.0 * M * N * K
            n_loop = min(20000, max(10, int(2.2 / b2b)))
            torch.cuda.synchronize()
            time.sleep(1.0)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n_loop):
                mx.mx_gemm(ea, sa, eb, sb, M, N, K, fa, fb, out=Cs[i & 1])
            b.record()
            torch.cuda.synchronize()
            sust = flops * n_loop / (a.elapsed_time(b) * 1e-3) / 1e12
            tf = flops / b2b / 1e12
            lines.append(f"| {label} | {flops / 1e9:.4g} | {med * 1e6:.1f} | {best * 1e6:.1f} | {b2b * 1e6:.1f} | {tf:.0f} | "
                         f"{100 * tf / fp8_burst:.1f} | {100 * tf / fp8_nom:.1f} | {sust:.0f} | {100 * sust / fp8_sust:.1f} |")
            del Cs
            torch.cuda.empty_cache()

    d1 = inputs.config1("cuda")
    gemm_row("C1 256x256x1024 E4M3 (latency-bound, no roofline claim)", d1["A"], d1["B"], 1, 0, 0, 0, 256, 256, 1024)
    ops3 = gemm_row("C3 8192x16384x4096 E4M3 x E4M3", d3["X"], d3["W"], 1, 0, 0, 0, 8192, 16384, 4096)
    n = 4096
    gemm_row("C4 forward 4096^3 E3M2 x E2M3", d4["X"], d4["W"], 1, 0, 2, 3, n, n, n, 1)
    gemm_row("C4 dgrad 4096^3 E3M2 x E2M3", d4["dY"], d4["W"], 1, 1, 2, 3, n, n, n, 1)
    gemm_row("C4 wgrad 4096^3 E3M2 x E3M2", d4["X"], d4["dY"], 0, 0, 2, 2, n, n, n, 1)
    gemm_row("C5 16384x28672x8192 E4M3 x E2M1", d5["X"], d5["W"], 1, 0, 0, 4, 16384, 28672, 8192)
    sustained_rows()

    # the oracle's dot products on a slab of C3, all host cores
    ea, sa, eb, sb = (t.cpu().numpy().reshape(-1) for t in ops3)
    Ms, Ns, K = 128, 1024, 4096
    t0 = time.perf_counter()
    O.gemm(ea[:Ms * K], sa[:Ms * K // 32], eb[:Ns * K], sb[:Ns * K // 32], Ms, Ns, K, 0, 0)
    dt = time.perf_counter() - t0
    gf = 2.0 * Ms * Ns * K / dt / 1e9
    lines += ["", "## Oracle on the host cores (reported baseline, not a target)", "",
              f"FP64 dot products of configuration 3 on a {Ms} x {Ns} x {K} slab: {dt:.2f} s on {O.threads()} threads = "
              f"{gf:.1f} GFLOP/s; the full 8192 x 16384 x 4096 product would take {2.0 * 8192 * 16384 * 4096 / gf / 1e9:.0f} s "
              "(extrapolated).  The quantize / dequantize sweep of the oracle is timed by the default run "
              "(`cpu_baseline` in the JSON line).", ""]
    return "\n".join(lines)


def run_cpu_baseline(rows: int = 2048, seconds_target: float = 15.0):
    """The oracle, as it stands, on the host cores: the same sweep on `rows` rows of the tensor."""
    import numpy as np
    import torch

    import oracle as O
    import workloads as inputs
    T = inputs.config2("cpu", rows, SWEEP_COLS, seed=2002)
    x = T.view(torch.int16).numpy().view(np.uint16)
    n = rows * SWEEP_COLS
    t0 = time.perf_counter()
    total = 0.0
    for fmt in range(6):
        e, s = O.quantize(x, 1, fmt, O.RNE, O.SWIZZLED)
        O.dequantize(e, s, rows, SWEEP_COLS, fmt, O.BF16, O.SWIZZLED)
        total += 2 * algorithmic_bytes(n, 2, FMT_BITS[fmt])
        if time.perf_counter() - t0 > 4 * seconds_target:
            break
    dt = time.perf_counter() - t0
    return {"value": total / dt / 1e9, "unit": "GB/s", "cores": O.threads(), "kind": "oracle",
            "sample": f"quantize+dequantize sweep, 6 formats, {rows}x{SWEEP_COLS} BF16 slice of the "
                      f"sweep tensor, {dt:.1f} s"}, dt


def main_ours(args, rank, world, local_rank):
    import torch

    import paper_2310_10537_b200 as mx
    import workloads as inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    peaks = measured_peaks()
    sampler = ClockSampler(local_rank) if rank == 0 else None  # polling by the time the timed region starts
    w = Workload(torch, mx, inputs, dev, seed_offset=rank)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        w.step()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(w.N_EVENTS)] for _ in range(args.steps)]
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    barrier()
    if sampler:
        sampler.begin()
    t_begin.record()
    for i in range(args.steps):
        w.step(evs[i])
    t_end.record()
    barrier()
    if sampler:
        sampler.end()
    clocks = sampler.stop() if sampler else None

    def phase(a, b):
        return sum(e[a].elapsed_time(e[b]) for e in evs) / args.steps  # ms per step

    ms = {"quantize_sweep": phase(0, 1), "dequantize_sweep": phase(1, 2), "quantize_x": phase(3, 4),
          "quantize_w_strided": phase(5, 6), "gemm": phase(7, 8)}
    ms_step = t_begin.elapsed_time(t_end) / args.steps
    ms_step_max, ms_sweep_max, ms_gemm_max, ms_q_max = max_over_ranks(
        [ms_step, ms["quantize_sweep"] + ms["dequantize_sweep"], ms["gemm"], ms["quantize_sweep"]], dev, world)
    if rank != 0:
        return

    value = job_throughput(w.bytes_sweep, world, ms_sweep_max * 1e-3) / 1e9
    gemm_tflops = job_throughput(w.flops, world, ms_gemm_max * 1e-3) / 1e12
    q_gbs = sum(w.bytes_q) / (ms["quantize_sweep"] * 1e-3) / 1e9
    fp8_peak = 2.0 * peaks["bf16_tflops"]
    line = {
        "metric": "mx_quantize_dequantize_GBps",
        "value": value,
        "unit": "GB/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": max(args.warmup, 3),
        "ms_per_step": ms_step_max,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "bf16->mx (fp8/fp6/fp4/int8 codes, e8m0 scales); gemm mxfp8 x mxfp8 -> f32",
        "data": "synthetic",
        "config": {
            "workload": "configs[1] quantize/dequantize sweep, BF16 8192x8192 Student-t(3)x4 with zero and "
                        "1e-30 blocks, six formats, k=32 along the last axis; plus configs[2] FFN "
                        "up-projection (quantize X, transposing quantize W, MXFP8 GEMM 8192x16384x4096)",
            "l2": "sweep inputs larger than L2 and read from alternating copies; a 512 MB read-only L2 flush "
                  "(evicts and writes back what the kernel before left) ahead of the sweep, of each FFN "
                  "quantize and of the GEMM, outside the phase timers",
            "rounding": "nearest-even", "scale_layout": "swizzled",
        },
        "phases_ms": ms,
        "gemm": {"metric": "mx_gemm_TFLOPs", "value": gemm_tflops, "unit": "TFLOP/s",
                 "workload": "configs[2] MXFP8 E4M3 8192x16384x4096, FP32 out",
                 "ms": ms_gemm_max},
        "quantize_x_GBps": w.bytes_qx / (ms["quantize_x"] * 1e-3) / 1e9,
        "quantize_w_strided_GBps": w.bytes_qw / (ms["quantize_w_strided"] * 1e-3) / 1e9,
        "dequantize_sweep_GBps": sum(w.bytes_q) / (ms["dequantize_sweep"] * 1e-3) / 1e9,
        "roofline": {
            "kernel": "quantize_lastaxis_kernel (six format instances, BF16 in, swizzled scales)",
            "bound": "hbm", "achieved": q_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": q_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
            "traffic": NCU_TRAFFIC.get("quantize"),
        },
        "roofline_gemm": {
            "kernel": "mx_gemm_pair_kernel (two-CTA 256x256 tiles, tcgen05 cta_group::2)", "bound": "tensor", "achieved": gemm_tflops / world,
            "peak": fp8_peak, "unit": "TFLOP/s", "frac": gemm_tflops / world / fp8_peak,
            "peak_source": f"2 x {peaks['source']} BF16 burst (nominal FP8:BF16 ratio)",
            "frac_of_sustained": gemm_tflops / world / (2.0 * peaks["bf16_tflops_sustained"]),
            "traffic": NCU_TRAFFIC.get("gemm"),
        },
        "gpu_launches": w.launches_per_step * args.steps,
        "clocks": clocks,
    }
    if world == 1:
        line["e2e"] = run_e2e(torch, mx, inputs, max(2, min(args.steps, 5)), 1)
        cpu, _ = run_cpu_baseline(rows=SWEEP_ROWS)
        line["cpu_baseline"] = cpu
        del w
        torch.cuda.empty_cache()
        line["other_configs"], per_config = run_extras(torch, mx, inputs, peaks, local_rank)
        line["roofline_gemm"]["per_config"] = per_config
        line["roofline_gemm"]["sustained"] = {k: v["sustained"] for k, v in per_config.items() if "sustained" in v}
    else:
        line["e2e"] = None
    print(json.dumps(line))


# DRAM read + write bytes per launch from the committed ncu captures (profiles/):
# quantize = one BF16 -> E4M3 launch on the sweep tensor (134.2 MB read + 42.6 MB written inside
# the kernel; the rest of the 69.2 MB output is still dirty in L2 when the kernel ends);
# gemm = captured on the 4096^3 case (37.4 + 22.4 MB) and scaled by bytes moved
# (A + B + scales + C: 640.7 MB for 8192 x 16384 x 4096 against 100.1 MB) -- DRAM traffic of the
# GEMM grows with the operand and output sizes, each read or written once.
NCU_TRAFFIC = {"quantize": 176.8e6, "gemm": 59.8e6 * 640.7 / 100.1}


def main_reference(args, rank, world):
    """The reference arm: the CPU oracle on the same metric, on a bounded sample per step."""
    if rank != 0:
        return
    times, total = [], None
    for i in range(max(args.warmup, 1) + args.steps):
        res, dt = run_cpu_baseline(rows=2048)
        if i >= max(args.warmup, 1):
            times.append(dt)
            total = res
    ms = 1e3 * sum(times) / len(times)
    # value over the timed steps
    rows = 2048
    nbytes = 2.0 * sum(algorithmic_bytes(rows * SWEEP_COLS, 2, b) for b in FMT_BITS)
    value = nbytes / (ms * 1e-3) / 1e9
    line = {
        "impl": "reference", "metric": "mx_quantize_dequantize_GBps", "value": value, "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64/int (CPU oracle)",
        "data": "synthetic",
        "config": {"workload": "configs[1] quantize/dequantize sweep; each step a 2048x8192 BF16 slice, "
                               "six formats, on the host cores"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": total["cores"], "kind": "oracle",
                         "sample": total["sample"]},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main_case(args):
    """A few launches of one kernel on a small case, for profiler captures (prints no bench line)."""
    import torch

    import paper_2310_10537_b200 as mx
    import workloads as inputs
    torch.cuda.set_device(0)
    reps = 3
    if args.case in ("quantize", "dequantize"):
        T = inputs.config2("cuda", SWEEP_ROWS, SWEEP_COLS)
        fmt = mx.FORMATS[args.fmt]
        e, s = mx.mx_quantize(T, 1, fmt)
        d = torch.empty_like(T)
        for _ in range(reps):
            if args.case == "quantize":
                mx.mx_quantize(T, 1, fmt, out=(e, s))
            else:
                mx.mx_dequantize(e, s, list(T.shape), fmt, torch.bfloat16, out=d)
    elif args.case == "quantize_strided":
        W = inputs.config3("cuda")["W"]
        fmt = mx.FORMATS[args.fmt]
        for _ in range(reps):
            mx.mx_quantize(W, 0, fmt)
    elif args.case == "gemm":
        n = 4096
        d = inputs.config4("cuda", n)
        fmt = mx.FORMATS[args.fmt]
        ea, sa = mx.mx_quantize(d["X"], 1, fmt)
        eb, sb = mx.mx_quantize(d["W"], 0, fmt)
        C = torch.empty((n, n), dtype=torch.float32, device="cuda")
        for _ in range(reps):
            mx.mx_gemm(ea, sa, eb, sb, n, n, n, fmt, fmt, out=C, check_status=True)
    elif args.case == "gemm_few_rows":  # a decode step: 16 activation rows against 16384 x 4096 weights (67 MB)
        M, N, K = 16, 16384, 4096
        g = torch.Generator(device="cuda").manual_seed(7)
        fmt = mx.FORMATS[args.fmt]
        ea, sa = mx.mx_quantize(torch.randn((M, K), generator=g, device="cuda", dtype=torch.bfloat16), 1, mx.MX_E4M3)
        eb, sb = mx.mx_quantize(torch.randn((N, K), generator=g, device="cuda", dtype=torch.bfloat16) * 0.05, 1, fmt)
        C = torch.empty((M, N), dtype=torch.float32, device="cuda")
        for _ in range(reps):
            mx.mx_gemm(ea, sa, eb, sb, M, N, K, mx.MX_E4M3, fmt, out=C, check_status=True)
    elif args.case == "gemm_dense":   # MXINT8 x MXINT8 through BF16: two dequantize launches + the dense GEMM
        n = 4096
        d = inputs.config4("cuda", n)
        ea, sa = mx.mx_quantize(d["X"], 1, mx.MX_INT8)
        eb, sb = mx.mx_quantize(d["W"], 0, mx.MX_INT8)
        C = torch.empty((n, n), dtype=torch.float32, device="cuda")
        ws = torch.empty(mx.mx_gemm_dense_workspace_bytes(n, n, n), dtype=torch.uint8, device="cuda")
        for _ in range(reps):
            mx.mx_gemm_dense(ea, sa, eb, sb, n, n, n, mx.MX_INT8, mx.MX_INT8, workspace=ws, out=C, check_status=True)
    elif args.case == "quantize_dual":
        T = inputs.config2("cuda", SWEEP_ROWS, SWEEP_COLS)
        fmt = mx.FORMATS[args.fmt]
        out = mx.mx_quantize_dual(T, fmt)
        for _ in range(reps):
            mx.mx_quantize_dual(T, fmt, out=out)
    elif args.case == "quantize_dual_f32":   # configuration 4's X (FP32 4096 x 4096, half-away rounding)
        T = inputs.config4("cuda")["X"]
        fmt = mx.FORMATS[args.fmt]
        out = mx.mx_quantize_dual(T, fmt, mx.MX_RHAZ)
        for _ in range(reps):
            mx.mx_quantize_dual(T, fmt, mx.MX_RHAZ, out=out)
    elif args.case == "conv":         # N 32, 56 x 56, C 256 -> 256, 3 x 3, padding 1: the operand fetched inside the GEMM
        x = torch.randn((32, 56, 56, 256), device="cuda", dtype=torch.bfloat16)
        wt = torch.randn((256, 3 * 3 * 256), device="cuda", dtype=torch.bfloat16) * 0.05
        fmt = mx.FORMATS[args.fmt]
        conv = mx.mx_conv_geometry(32, 56, 56, 256, 3, 3, (1, 1), (1, 1), (1, 1))
        ex, sx = mx.mx_quantize(x, 3, fmt)
        ew, sw = mx.mx_quantize(wt, 1, fmt)
        y = torch.empty((32 * 56 * 56, 256), dtype=torch.float32, device="cuda")
        for _ in range(reps):
            mx.mx_conv2d(ex, sx, ew, sw, conv, 256, fmt, fmt, out=y, check_status=True)
    elif args.case == "im2col":       # N 32, 56 x 56, C 256, 3 x 3, padding 1: 231 MB of E4M3 codes out
        x = torch.randn((32, 56, 56, 256), device="cuda", dtype=torch.bfloat16)
        fmt = mx.FORMATS[args.fmt]
        conv = mx.mx_conv_geometry(32, 56, 56, 256, 3, 3, (1, 1), (1, 1), (1, 1))
        ex, sx = mx.mx_quantize(x, 3, fmt)
        for _ in range(reps):
            mx.mx_im2col(ex, sx, conv, fmt)
    torch.cuda.synchronize()
    print(json.dumps({"case": args.case, "fmt": args.fmt, "launches": reps}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", choices=["step", "quantize", "dequantize", "quantize_strided", "gemm", "gemm_dense",
                                       "gemm_few_rows", "quantize_dual", "quantize_dual_f32", "im2col", "conv"],
                    default="step", help="'step' = the benchmark; the others run three launches of one "
                                         "kernel on a small case for a profiler capture")
    ap.add_argument("--fmt", choices=FMT_NAMES, default="e4m3")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--report", action="store_true", help="per-kernel protocol on every configuration, as markdown "
                                                          "on stdout (one GPU, a few minutes)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.report:
        import torch

        import paper_2310_10537_b200 as mx
        import workloads as inputs
        torch.cuda.set_device(0)
        print("# Per-kernel measurements on one B200 (`python bench.py --report`)\n")
        print(run_report(torch, mx, inputs))
    elif args.case != "step":
        main_case(args)
    elif args.impl == "reference":
        main_reference(args, rank, world)
    else:
        main_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
