#!/usr/bin/env python
"""Benchmark of the im2win hot path on B200.

One STEP = the whole path on one batch: im2win transform (NCHW input -> im2win tensor in the
workspace) followed by the im2win-based convolution on the tensor cores (`im2win_conv` with the
untransformed input as source).  The default workload is the ResNet-style 3x3 layer of the benchmark
definition (N=128, C=64, 58x58 pre-padded, K=64, stride 1) with seeded synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--mode tf32|bf16] [--workload NAME]
    python bench.py --impl reference      # the CPU oracle timed on the host cores
    python bench.py --sweep               # every named layer, one JSON line each on stderr

Prints ONE JSON line on stdout (rank 0).  Timing: CUDA events on the launching stream around each
step, L2 flushed (untimed) before every step, barrier + synchronize around the timed region, max over
ranks.  With N > 1 every rank runs its own batch (images are independent, no collective on the data
path): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2306_14320_b200 import workloads as wl  # noqa: E402

METRIC = "conv TFLOP/s (transform + im2win convolution, FLOPs = 2*N*K*Ho*Wo*C*Fh*Fw)"
UNIT = "TFLOP/s"
NOMINAL_TF32_OVER_BF16 = 1.1 / 2.25
# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (conv_tc_persistent__*.md)
# (conv_tc_persistent__*.md, conv_tc_strip__*.md): the kernel the library chooses for that workload
NCU_TRAFFIC_BYTES = {("resnet3x3", "tf32"): 319.52e6 + 83.52e6, ("stem7x7", "tf32"): 277.09e6 + 352.88e6,
                     ("down3x3", "tf32"): 322.35e6 + 74.64e6,
                     ("deep3x3", "tf32"): 90.54e6 + 4.44e6, ("deep3x3", "bf16"): 89.36e6 + 3.78e6}
KERNEL_NAMES = {1: "conv_tc_strip_kernel", 2: "conv_tc_persistent_kernel", 3: "conv_tc_kernel", 4: "conv_fp32_kernel",
                5: "conv_tc_window_kernel"}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def measure_matmul_peaks(torch, sustained_s: float = 4.0):
    """Dense matmul throughput of this GPU through torch (cuBLAS), 8192^3, outside every timed region:
    TF32 (fp32 operands, allow_tf32) and BF16, each as the best of 10 and as a back-to-back loop of
    `sustained_s` seconds (the power cap pulls the clock down within a second or two)."""
    out = {}
    n = 8192
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        for name, dt in (("tf32", torch.float32), ("bf16", torch.bfloat16)):
            a = torch.randn(n, n, device="cuda", dtype=dt)
            b_ = torch.randn(n, n, device="cuda", dtype=dt)
            c = torch.empty(n, n, device="cuda", dtype=dt)
            for _ in range(3):
                torch.matmul(a, b_, out=c)
            best = None
            for _ in range(10):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); torch.matmul(a, b_, out=c); e1.record(); torch.cuda.synchronize()
                t = e0.elapsed_time(e1)
                best = t if best is None or t < best else best
            out[f"{name}_tflops"] = 2.0 * n ** 3 / best / 1e9
            if sustained_s > 0:
                reps = max(10, int(sustained_s * 1e3 / best))
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    torch.matmul(a, b_, out=c)
                e1.record(); torch.cuda.synchronize()
                out[f"{name}_tflops_sustained"] = 2.0 * n ** 3 * reps / e0.elapsed_time(e1) / 1e9
            del a, b_, c
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    out["how"] = f"torch.matmul {n}^3 (2*n^3 FLOPs), best of 10 and back to back for {sustained_s:g} s; TF32 = fp32 operands with allow_tf32"
    return out


def time_conv_only(layer, mode_name, steps, torch, b, flush_buf):
    """Convolution from a pre-built im2win tensor only (CUDA events, L2 flushed between iterations)."""
    mode = {"tf32": b.MODE_TF32, "bf16": b.MODE_BF16}[mode_name]
    dims = layer.dims()
    ho, wo = b.out_dims(dims)
    ws_bytes = b.workspace_bytes(dims)
    x = torch.from_numpy(wl.make_input(layer)).cuda()
    f = torch.from_numpy(wl.make_filter(layer)).cuda()
    ws_all = torch.empty(max(ws_bytes, b.conv_workspace_bytes(dims, b.SRC_NCHW, mode)) // 4, dtype=torch.float32, device="cuda")
    ws = ws_all[:ws_bytes // 4]
    off = (ws_bytes + 255) // 256 * 256 // 4
    scratch = ws_all[off:] if ws_all.numel() > off else None
    out = torch.empty((layer.N, layer.K, ho, wo), dtype=torch.float32, device="cuda")
    b.transform(x, dims, ws)
    for _ in range(3):
        b.conv(ws, b.SRC_IM2WIN, f, dims, mode, out, scratch)
    ts = []
    for _ in range(steps):
        flush_buf.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); b.conv(ws, b.SRC_IM2WIN, f, dims, mode, out, scratch); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    if b.last_device_status() != 0:
        raise RuntimeError("device status word set")
    return {"ms": sum(ts) / len(ts), "ms_best_of_5": min(ts[:5]), "tflops": _flops(layer, ho, wo) / (sum(ts) / len(ts)) / 1e9}


def kernel_used(layer, mode_name, torch, b):
    """Name of the convolution kernel the library chooses for this workload: one untimed call through the
    test build of the same object files (the only build that records its choice), default switches."""
    mode = {"tf32": b.MODE_TF32, "bf16": b.MODE_BF16}[mode_name]
    dims = layer.dims()
    ho, wo = b.out_dims(dims)
    try:
        b.use_test_library(True)
        ws = torch.zeros(b.conv_workspace_bytes(dims, b.SRC_NCHW, mode) // 4 + 64, dtype=torch.float32, device="cuda")
        x = torch.zeros((layer.N, layer.C, layer.H, layer.W), dtype=torch.float32, device="cuda")
        f = torch.zeros((layer.K, layer.C, layer.Fh, layer.Fw), dtype=torch.float32, device="cuda")
        out = torch.empty((layer.N, layer.K, ho, wo), dtype=torch.float32, device="cuda")
        b.conv(x, b.SRC_NCHW, f, dims, mode, out, ws)
        torch.cuda.synchronize()
        return KERNEL_NAMES.get(b.last_kernel(), "unknown")
    except (ImportError, OSError, RuntimeError, AttributeError):
        return "unknown"
    finally:
        b.use_test_library(False)


def _flops(layer, ho, wo):
    return 2.0 * layer.N * layer.K * ho * wo * layer.C * layer.Fh * layer.Fw


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self._stop = [], set(), threading.Event()
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": "nvmlClocksEventReasonHwSlowdown", "hw_thermal_slowdown": "nvmlClocksEventReasonHwThermalSlowdown",
                 "sw_thermal_slowdown": "nvmlClocksEventReasonSwThermalSlowdown", "sw_power_cap": "nvmlClocksEventReasonSwPowerCap"}
        alt = {"hw_slowdown": "nvmlClocksThrottleReasonHwSlowdown", "hw_thermal_slowdown": "nvmlClocksThrottleReasonHwThermalSlowdown",
               "sw_thermal_slowdown": "nvmlClocksThrottleReasonSwThermalSlowdown", "sw_power_cap": "nvmlClocksThrottleReasonSwPowerCap"}
        masks = {k: getattr(nv, v, getattr(nv, alt[k], 0)) for k, v in names.items()}
        get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = get(self.h)
                for k, m in masks.items():
                    if m and (r & m):
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv:
            self.t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self.nv:
            self.t.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        return {"sm_mhz": float(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _cpu_baseline(layer, seconds_target=12.0):
    """The oracle as it stands (Algorithm 1 then Algorithm 2 in double), on a bounded sample of images."""
    import oracle
    f = wl.make_filter(layer)
    one = layer.with_batch(1)
    x1 = wl.make_input(layer, slice(0, 1))
    sh1 = oracle.Shape(*one.dims())
    t0 = time.perf_counter()
    oracle.conv_via_im2win(oracle.im2win(x1, sh1), f, sh1)
    t1 = time.perf_counter() - t0
    n = int(max(1, min(layer.N, seconds_target / max(t1, 1e-6))))
    sub = layer.with_batch(n)
    x = wl.make_input(layer, slice(0, n))
    shn = oracle.Shape(*sub.dims())
    t0 = time.perf_counter()
    oracle.conv_via_im2win(oracle.im2win(x, shn), f, shn)
    dt = time.perf_counter() - t0
    ho, wo = oracle.out_dims(shn)
    return {"value": _flops(sub, ho, wo) / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n} of {layer.N} images of {layer.name}: Algorithm 1 + Algorithm 2, fp64 accumulation, {dt:.2f} s"}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    layer = wl.CONFIGS[args.workload]
    f = wl.make_filter(layer)
    n = max(1, min(layer.N, args.ref_images))
    sub = layer.with_batch(n)
    x = wl.make_input(layer, slice(0, n))
    sh = oracle.Shape(*sub.dims())
    ho, wo = oracle.out_dims(sh)
    for _ in range(args.warmup):
        oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.conv_via_im2win(oracle.im2win(x, sh), f, sh)
    dt = (time.perf_counter() - t0) / args.steps
    val = _flops(sub, ho, wo) / dt / 1e12
    sample = f"{n} of {layer.N} images of {layer.name} per step: Algorithm 1 + Algorithm 2, fp64 accumulation"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": layer.name, "dims_NCHWKFhFws": list(layer.dims()), "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def time_layer(layer, mode_name, steps, warmup, torch, b, flush_buf, sampler_index=None, e2e=True):
    """Times transform, conv and the whole step for one layer on the current device."""
    mode = {"tf32": b.MODE_TF32, "bf16": b.MODE_BF16}[mode_name]
    dims = layer.dims()
    ho, wo = b.out_dims(dims)
    ws_bytes, col_bytes = b.workspace_bytes(dims), b.im2col_bytes(dims)
    x_host = torch.from_numpy(wl.make_input(layer)).pin_memory()
    f_host = torch.from_numpy(wl.make_filter(layer)).pin_memory()
    x, f = x_host.cuda(), f_host.cuda()
    # one workspace: the im2win tensor, then (from the next 256-byte boundary) scratch for the filter
    # copy some kernels stream; sized by the library's own query
    ws_total = max(ws_bytes, b.conv_workspace_bytes(dims, b.SRC_NCHW, mode))
    ws_all = torch.empty(ws_total // 4, dtype=torch.float32, device="cuda")
    ws = ws_all[:ws_bytes // 4]
    scratch_off = (ws_bytes + 255) // 256 * 256 // 4
    scratch = ws_all[scratch_off:] if ws_all.numel() > scratch_off else None
    out = torch.empty((layer.N, layer.K, ho, wo), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def step(events=None):
        if events:
            events[0].record(stream)
        b.transform(x, dims, ws)
        if events:
            events[1].record(stream)
        b.conv(ws, b.SRC_IM2WIN, f, dims, mode, out, scratch)
        if events:
            events[2].record(stream)

    for _ in range(warmup):
        flush_buf.zero_()
        step()
    torch.cuda.synchronize()
    if b.last_device_status() != 0:
        raise RuntimeError("device status word set during warm-up")
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    if sampler:
        sampler.__enter__()
    t_wall0 = time.perf_counter()
    for k in range(steps):
        flush_buf.zero_()  # L2 flush, outside the event-timed interval
        step(evs[k])
    torch.cuda.synchronize()
    t_wall = time.perf_counter() - t_wall0
    if sampler:
        sampler.__exit__()
    if b.last_device_status() != 0:
        raise RuntimeError("device status word set during the timed region")
    # The same K steps once more with no event record between the two kernels: the convolution kernel is a
    # programmatic dependent of the transform kernel, and its prologue overlaps that kernel's tail only when
    # nothing sits between them in the stream.  Reported beside the timed region's figure, not instead of it.
    evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
    for k in range(steps):
        flush_buf.zero_()
        evs2[k][0].record(stream)
        step()
        evs2[k][1].record(stream)
    torch.cuda.synchronize()
    if b.last_device_status() != 0:
        raise RuntimeError("device status word set during the back-to-back steps")
    t_bb = [e[0].elapsed_time(e[1]) for e in evs2]
    t_tr = [e[0].elapsed_time(e[1]) for e in evs]
    t_cv = [e[1].elapsed_time(e[2]) for e in evs]
    t_st = [e[0].elapsed_time(e[2]) for e in evs]
    res = {
        "ms_step": sum(t_st) / steps, "ms_transform": sum(t_tr) / steps, "ms_conv": sum(t_cv) / steps,
        "ms_step_best": min(t_st), "ms_transform_best": min(t_tr), "ms_conv_best": min(t_cv),
        "ms_step_back_to_back": sum(t_bb) / steps,
        # the paper's protocol (Section IV-B): five runs, the best kept; and the median of twenty
        "ms_step_best_of_5": min(t_st[:5]), "ms_step_median_of_20": float(statistics.median(t_st[:20])),
        "ms_conv_best_of_5": min(t_cv[:5]), "ms_conv_median_of_20": float(statistics.median(t_cv[:20])),
        "wall_s": t_wall, "flops": _flops(layer, ho, wo), "workspace_bytes": ws_bytes, "im2col_bytes": col_bytes,
        "filter_scratch_bytes": ws_total - ws_bytes,
        "bytes_in": x.numel() * 4, "bytes_f": f.numel() * 4, "bytes_out": out.numel() * 4,
        "clocks": sampler.summary() if sampler else None,
    }
    # algorithmic bytes: the transform reads each needed input row once and writes each strip once;
    # the conv reads the im2win tensor and the filter once and writes the output once
    h_used = (ho - 1) * layer.s + layer.Fh
    res["transform_bytes"] = 4.0 * layer.N * layer.C * (h_used * layer.W) + ws_bytes
    res["conv_bytes"] = float(ws_bytes + res["bytes_f"] + res["bytes_out"])
    # the fused source kind: same result straight from the untransformed input, no im2win tensor in HBM
    try:
        for _ in range(3):
            b.conv(x, b.SRC_NCHW_FUSED, f, dims, mode, out, scratch)
        fe = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for k in range(steps):
            flush_buf.zero_()
            fe[k][0].record(stream)
            b.conv(x, b.SRC_NCHW_FUSED, f, dims, mode, out, scratch)
            fe[k][1].record(stream)
        torch.cuda.synchronize()
        if b.last_device_status() != 0:
            raise RuntimeError("device status word set during the fused timing")
        tf_ = [e[0].elapsed_time(e[1]) for e in fe]
        res["ms_fused"], res["ms_fused_best"] = sum(tf_) / steps, min(tf_)
        res["fused_bytes"] = float(res["bytes_in"] + res["bytes_f"] + res["bytes_out"])
    except b.Im2winError as exc:
        if exc.code != b.EUNSUPPORTED:
            raise
        res["ms_fused"] = None
    # the bf16 OUTPUT variant (im2win_conv_bf16out from the im2win tensor): halves the output write
    res["ms_conv_bf16out"] = None
    try:
        out16 = torch.empty(layer.N * layer.K * ho * wo, dtype=torch.int16, device="cuda")
        for _ in range(3):
            b.conv_bf16out(ws, b.SRC_IM2WIN, f, dims, mode, out16, scratch)
        oe = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for k in range(steps):
            flush_buf.zero_()
            oe[k][0].record(stream)
            b.conv_bf16out(ws, b.SRC_IM2WIN, f, dims, mode, out16, scratch)
            oe[k][1].record(stream)
        torch.cuda.synchronize()
        if b.last_device_status() != 0:
            raise RuntimeError("device status word set during the bf16-output timing")
        res["ms_conv_bf16out"] = sum(e[0].elapsed_time(e[1]) for e in oe) / steps
        del out16
    except b.Im2winError as exc:
        if exc.code != b.EUNSUPPORTED:
            raise
    # the NHWC output variant (im2win_conv_nhwc from the im2win tensor): same bytes, channels-last stores
    res["ms_conv_nhwc"] = None
    try:
        for _ in range(3):
            b.conv_nhwc(ws, b.SRC_IM2WIN, f, dims, mode, out, scratch)
        ne = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        for k in range(steps):
            flush_buf.zero_()
            ne[k][0].record(stream)
            b.conv_nhwc(ws, b.SRC_IM2WIN, f, dims, mode, out, scratch)
            ne[k][1].record(stream)
        torch.cuda.synchronize()
        if b.last_device_status() != 0:
            raise RuntimeError("device status word set during the NHWC-output timing")
        res["ms_conv_nhwc"] = sum(e[0].elapsed_time(e[1]) for e in ne) / steps
    except b.Im2winError as exc:
        if exc.code != b.EUNSUPPORTED:
            raise
    # the bf16 storage variant of the im2win tensor: always a BF16-mode convolution, whatever the line's mode
    res["ms_transform_bf16"] = res["ms_conv_bf16src"] = None
    if True:
        ws16 = torch.empty(b.workspace_bytes_bf16(dims) // 2, dtype=torch.int16, device="cuda")
        n16 = b.conv_workspace_bytes(dims, b.SRC_IM2WIN_BF16, b.MODE_BF16)
        scratch16 = torch.empty(n16 // 4 + 64, dtype=torch.float32, device="cuda") if n16 else None
        try:
            for _ in range(3):
                b.transform_bf16(x, dims, ws16)
                b.conv(ws16, b.SRC_IM2WIN_BF16, f, dims, b.MODE_BF16, out, scratch16)
            be = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
            for k in range(steps):
                flush_buf.zero_()
                be[k][0].record(stream)
                b.transform_bf16(x, dims, ws16)
                be[k][1].record(stream)
                b.conv(ws16, b.SRC_IM2WIN_BF16, f, dims, b.MODE_BF16, out, scratch16)
                be[k][2].record(stream)
            torch.cuda.synchronize()
            if b.last_device_status() != 0:
                raise RuntimeError("device status word set during the bf16-storage timing")
            res["ms_transform_bf16"] = sum(e[0].elapsed_time(e[1]) for e in be) / steps
            res["ms_conv_bf16src"] = sum(e[1].elapsed_time(e[2]) for e in be) / steps
        except b.Im2winError as exc:
            if exc.code != b.EUNSUPPORTED:
                raise
        del ws16
    if e2e:
        out_host = torch.empty((layer.N, layer.K, ho, wo), dtype=torch.float32).pin_memory()
        n_e2e = max(3, min(steps, 10))
        for _ in range(2):
            b.conv_host(x_host, f_host, dims, mode, out_host)
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            b.conv_host(x_host, f_host, dims, mode, out_host)
        res["e2e_s"] = (time.perf_counter() - t0) / n_e2e
        b.host_release()
    return res


def max_over_ranks(values, dist, device="cpu"):
    """Element-wise maximum of a list of per-rank timings over all ranks (the slowest rank defines the
    job's time); identity when torch.distributed is not initialised.  Used for every multi-GPU number."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def job_value(flops_per_rank, world, ms_step_max):
    """Whole-job TFLOP/s under weak scaling: every rank did `flops_per_rank` in the slowest rank's time."""
    return world * flops_per_rank / ms_step_max / 1e9


def run_gpu(args):
    import torch
    from paper_2306_14320_b200 import binding as b, build
    build.build_library()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = _peaks()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    matmul_peaks = None
    if rank == 0 and not args.sweep and not args.no_matmul_peaks:
        matmul_peaks = measure_matmul_peaks(torch, args.peak_seconds)

    if args.sweep:
        if args.sweep == "all":
            names = [n for n in wl.CONFIGS if not n.startswith("table1_")]
        elif args.sweep == "table1":
            names = [l.name for l in wl.TABLE_I_LAYERS]
        else:
            names = args.sweep.split(",")
        for name in names:
            for n_batch in ([128] if not args.sweep_batches else [int(v) for v in args.sweep_batches.split(",")]):
                layer = wl.CONFIGS[name]
                layer = layer.with_batch(min(n_batch, layer.N) if name == "tiny" else n_batch)
                for mode in ("tf32", "bf16"):
                    r = time_layer(layer, mode, args.steps, args.warmup, torch, b, flush_buf, None, e2e=False)
                    peak = peaks["bf16_tflops"] * (NOMINAL_TF32_OVER_BF16 if mode == "tf32" else 1.0)
                    line = {"layer": layer.name, "N": layer.N, "dims": list(layer.dims()), "mode": mode,
                            "conv_tflops": r["flops"] / r["ms_conv"] / 1e9, "conv_tflops_best": r["flops"] / r["ms_conv_best"] / 1e9,
                            "conv_frac_tensor_peak": r["flops"] / r["ms_conv"] / 1e9 / peak,
                            "conv_gbs": r["conv_bytes"] / r["ms_conv"] / 1e6, "conv_frac_hbm": r["conv_bytes"] / r["ms_conv"] / 1e6 / peaks["hbm_gbs"],
                            "transform_gbs": r["transform_bytes"] / r["ms_transform"] / 1e6,
                            "transform_frac_hbm": r["transform_bytes"] / r["ms_transform"] / 1e6 / peaks["hbm_gbs"],
                            "step_tflops": r["flops"] / r["ms_step"] / 1e9, "ms_conv": r["ms_conv"], "ms_transform": r["ms_transform"],
                            "workspace_bytes": r["workspace_bytes"], "im2col_bytes": r["im2col_bytes"], "peaks": peaks["source"],
                            "ms_transform_bf16": r.get("ms_transform_bf16"), "ms_conv_bf16src": r.get("ms_conv_bf16src"),
                            "ms_conv_bf16out": r.get("ms_conv_bf16out"), "ms_conv_nhwc": r.get("ms_conv_nhwc"),
                            "ms_fused": r.get("ms_fused"),
                            "fused_tflops": (r["flops"] / r["ms_fused"] / 1e9) if r.get("ms_fused") else None,
                            "fused_frac_hbm": (r["fused_bytes"] / r["ms_fused"] / 1e6 / peaks["hbm_gbs"]) if r.get("ms_fused") else None}
                    print(json.dumps(line), file=sys.stderr, flush=True)
        return

    layer = wl.CONFIGS[args.workload]
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    r = time_layer(layer, args.mode, args.steps, args.warmup, torch, b, flush_buf, local, e2e=True)
    torch.cuda.synchronize()
    ms_step, ms_e2e, ms_conv, ms_tr, ms_bb = max_over_ranks(
        [r["ms_step"], r["e2e_s"] * 1e3, r["ms_conv"], r["ms_transform"], r["ms_step_back_to_back"]], dist, device="cuda")
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    flops = r["flops"]
    value = job_value(flops, world, ms_step)
    tensor_peak = peaks["bf16_tflops"] * (NOMINAL_TF32_OVER_BF16 if args.mode == "tf32" else 1.0)
    t_hbm = r["conv_bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tensor = flops / (tensor_peak * 1e12)
    if t_hbm >= t_tensor:
        roof = {"bound": "hbm", "achieved": r["conv_bytes"] / ms_conv / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": flops / ms_conv / 1e9, "peak": tensor_peak, "unit": "TFLOP/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = args.traffic if args.traffic is not None else NCU_TRAFFIC_BYTES.get((layer.name, args.mode))
    roof["kernel"] = kernel_used(layer, args.mode, torch, b)
    roof["peak_source"] = f"of {peaks['source']}" + (" (bf16 burst x nominal tf32/bf16 ratio)" if roof["bound"] == "tensor" and args.mode == "tf32" else "")
    roof["algorithmic_bytes_per_launch"] = r["conv_bytes"]
    roof["kernel_ms"] = ms_conv
    roof["conv_tflops"] = flops / ms_conv / 1e9
    roof["conv_frac_tensor_peak"] = flops / ms_conv / 1e9 / tensor_peak

    if matmul_peaks:
        key = "tf32_tflops" if args.mode == "tf32" else "bf16_tflops"
        roof["conv_frac_measured_matmul"] = roof["conv_tflops"] / matmul_peaks[key]
    # the tensor-bound layers of the benchmark definition, convolution only (not part of `value`)
    extra = {}
    if world == 1 and not args.no_extra_layers:
        for name in ("deep3x3", "sweep_L5", "sweep_L10", "sweep_L4", "sweep_L2"):
            extra[name] = {}
            for m in ("tf32", "bf16"):
                r2 = time_conv_only(wl.CONFIGS[name], m, 10, torch, b, flush_buf)
                pk = peaks["bf16_tflops"] * (NOMINAL_TF32_OVER_BF16 if m == "tf32" else 1.0)
                r2["frac_tensor_peak"] = r2["tflops"] / pk
                if matmul_peaks:
                    r2["frac_measured_matmul"] = r2["tflops"] / matmul_peaks[f"{m}_tflops"]
                r2["kernel"] = kernel_used(wl.CONFIGS[name], m, torch, b)
                extra[name][m] = r2
    cpu = _cpu_baseline(layer) if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": args.mode, "data": "synthetic",
        "ms_per_step_best_of_5": r["ms_step_best_of_5"], "ms_per_step_median_of_20": r["ms_step_median_of_20"],
        "value_best_of_5": job_value(flops, world, r["ms_step_best_of_5"]),
        "value_median_of_20": job_value(flops, world, r["ms_step_median_of_20"]),
        "back_to_back": {"ms_per_step": ms_bb, "value": job_value(flops, world, ms_bb),
                         "how": "the same K steps again with no event record between the transform and the convolution: "
                                "the convolution kernel is launched as a programmatic dependent of the transform kernel and "
                                "sets up while that kernel drains; `value` keeps the record in between"},
        "config": {"workload": layer.name, "dims_NCHWKFhFws": list(layer.dims()), "batch_per_gpu": layer.N,
                   "parallelism": f"dp{world} (independent batches, no collective)",
                   "l2": "flushed before every step by a 256 MiB write outside the event-timed interval; "
                         "the step's own working set is 532 MB",
                   "timing": "CUDA events on the launching stream around each step, mean over steps"},
        "roofline": roof,
        "transform": {"gbs": r["transform_bytes"] / ms_tr / 1e6, "frac_hbm": r["transform_bytes"] / ms_tr / 1e6 / peaks["hbm_gbs"],
                      "ms": ms_tr, "algorithmic_bytes": r["transform_bytes"], "peak_source": f"of {peaks['source']}"},
        "workspace_bytes": r["workspace_bytes"], "im2col_bytes": r["im2col_bytes"],
        "filter_scratch_bytes": r["filter_scratch_bytes"],
        "matmul_peaks_measured": matmul_peaks,
        "tensor_bound_layers": extra or None,
        "fused": ({"value": world * flops / r["ms_fused"] / 1e9, "unit": UNIT, "ms": r["ms_fused"],
                   "what": "im2win_conv with src_kind NCHW_FUSED: same result from the untransformed input in one kernel, "
                           "no im2win tensor written (workspace 0 bytes); not part of `value`",
                   "frac_hbm": r["fused_bytes"] / r["ms_fused"] / 1e6 / peaks["hbm_gbs"]} if r.get("ms_fused") else None),
        "bf16_storage": ({"ms_transform": r["ms_transform_bf16"], "ms_conv": r["ms_conv_bf16src"],
                          "what": "the im2win tensor stored as bf16 (im2win_transform_bf16, src_kind IM2WIN_BF16): "
                                  "half the workspace; a BF16-mode convolution whatever this line's mode; not part of `value`"}
                         if r.get("ms_conv_bf16src") else None),
        "bf16_output": ({"ms_conv": r["ms_conv_bf16out"],
                         "what": "im2win_conv_bf16out: the same convolution with the result stored as bf16 "
                                 "(half the output write); not part of `value`"} if r.get("ms_conv_bf16out") else None),
        "nhwc_output": ({"ms_conv": r["ms_conv_nhwc"],
                         "what": "im2win_conv_nhwc: the same convolution with the fp32 result written N x Ho x Wo x K; "
                                 "not part of `value`"} if r.get("ms_conv_nhwc") else None),
        "e2e": {"value": world * flops / ms_e2e / 1e9, "unit": UNIT, "h2d_bytes_per_step": r["bytes_in"] + r["bytes_f"],
                "d2h_bytes_per_step": r["bytes_out"], "ms_per_step": ms_e2e,
                "how": "im2win_conv_host: pinned host buffers in, pinned host buffer out, wall clock per call; the call "
                       "pipelines the batch in eight chunks through three streams and runs the FUSED source kind on each "
                       "(no im2win tensor in memory), so the transform kernel is not part of this figure"},
        "gpu_launches": 2 * args.steps,
        "clocks": r["clocks"],
    }
    if cpu:
        line["cpu_baseline"] = cpu
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--mode", default="tf32", choices=["tf32", "bf16"])
    ap.add_argument("--workload", default="resnet3x3", choices=list(wl.CONFIGS))
    ap.add_argument("--sweep", nargs="?", const="all", default=None, help="per-layer lines on stderr instead of the bench line")
    ap.add_argument("--sweep-batches", default=None)
    ap.add_argument("--traffic", type=float, default=None, help="DRAM bytes per conv launch from an ncu capture (profiles/)")
    ap.add_argument("--ref-images", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-matmul-peaks", action="store_true")
    ap.add_argument("--no-extra-layers", action="store_true")
    ap.add_argument("--peak-seconds", type=float, default=4.0, help="length of the sustained matmul loops")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as plain `python bench.py --gpus N`: become N ranks on this node (one per GPU)
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
        os.execv(sys.executable, cmd)
    if args.warmup < 3 and args.impl == "b200":
        args.warmup = 3
    if args.impl == "reference":
        if args.steps == 200:
            args.steps = 5
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
