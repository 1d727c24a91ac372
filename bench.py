#!/usr/bin/env python
"""Benchmark of the fused operator chains on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

One step = one pass of the headline chain over one batch of synthetic input: config 2,
bf16 Y = 0.5*GELU_tanh(X W^T + b) + R with X[8192,4096], W[4096,4096] (fp32 accumulate, bf16 out),
through the C-ABI call kf_gemm_epilogue.  The metric is fused-chain TFLOP/s (2*M*N*K per call).
With N > 1 (torchrun) every rank runs the same shape on its own batch (rows are independent:
weak scaling, no collective on the data path); the value is the aggregate over ranks and the
time is the maximum over ranks.

Prints ONE JSON line with the metric, the roofline of the dominant kernel, the CPU oracle
timed on a bounded sample (rank 0, N = 1), the end-to-end figure with host buffers, and, as
context, every other benchmark chain next to the same chain as separate torch ops.

--impl reference times the fp64 CPU oracle on the host cores instead (a deliberately slow
program: a reported baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import kf_inputs as ki  # noqa: E402

WORKLOAD = "c2"
M2, N2, K2 = 8192, 4096, 4096
FLOPS_C2 = 2.0 * M2 * N2 * K2
ALG_BYTES_C2 = 2 * (M2 * K2 + N2 * K2 + N2 + 2 * M2 * N2)   # X, W, b, R read once, Y written once
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            d["_source"] = "measured"
            return d
        except Exception:
            pass
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def c2_traffic_bytes():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the config-2 kernel: the figure the
    committed ncu summary of that kernel states (a line `dram_bytes_per_launch = N`), or None."""
    path = os.path.join(ROOT, "profiles", "umma_chain_kernel_c2_gelu_residual.md")
    try:
        for line in open(path):
            if line.strip().startswith("dram_bytes_per_launch"):
                return float(line.split("=")[1].split()[0])
    except Exception:
        pass
    return None


# ------------------------------------------------------------------ clocks during the timed region
class ClockSampler:
    """Polls NVML (read-only) for SM clock and throttle reasons while a timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------ multi-rank bookkeeping
def max_over_ranks(ms: float, world: int, device=None) -> float:
    """The slowest rank's time: what the whole job took (any torch.distributed backend)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank_per_step: float, world: int, ms_per_step: float) -> float:
    """Aggregate throughput of `world` replicas that each did the full per-rank work."""
    return flops_per_rank_per_step * world / (ms_per_step * 1e-3) / 1e12


def rank_seed(rank: int) -> int:
    """Each rank generates its own batch: the seed is the rank."""
    return int(rank)


# ------------------------------------------------------------------ helpers
def to_dev(a, device):
    import torch
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(a).to(device)


def to_pinned(a):
    import torch
    if a.dtype == np.uint16:
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(a)
    return t.pin_memory()


def time_calls_stats(fn, iters, warmup, graph_batch=0, flush=None):
    """Device time of fn() in microseconds: {"mean", "median", "min", "samples"} over CUDA-event pairs
    on the current stream, one pair per call (per graph replay when graph_batch > 0).

    graph_batch > 0 captures that many calls into a CUDA graph first, so that launch-bound
    chains are timed on the device rather than at the host's launch rate.  flush: a callable run
    before every timed sample, outside its event pair (the cold-cache variant writes a buffer
    larger than L2 there)."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    runner, per = fn, 1
    if graph_batch > 0:
        try:
            g = torch.cuda.CUDAGraph()
            s = torch.cuda.Stream()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                fn()
                with torch.cuda.graph(g, stream=s):
                    for _ in range(graph_batch):
                        fn()
            torch.cuda.current_stream().wait_stream(s)
            torch.cuda.synchronize()
            runner, per = g.replay, graph_batch
            runner()
            torch.cuda.synchronize()
        except Exception:
            runner, per = fn, 1
    reps = max(3, iters // per)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for e0, e1 in pairs:
        if flush is not None:
            flush()
        e0.record()
        runner()
        e1.record()
    torch.cuda.synchronize()
    t = np.array([e0.elapsed_time(e1) * 1e3 / per for e0, e1 in pairs])
    return {"mean": float(t.mean()), "median": float(np.median(t)), "min": float(t.min()), "samples": int(reps)}


def time_calls(fn, iters, warmup, graph_batch=0):
    """Average device time of fn() in microseconds over back-to-back calls (one event pair around
    all of them: what a loop of calls costs per call)."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    runner, per = fn, 1
    if graph_batch > 0:
        try:
            g = torch.cuda.CUDAGraph()
            s = torch.cuda.Stream()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                fn()
                with torch.cuda.graph(g, stream=s):
                    for _ in range(graph_batch):
                        fn()
            torch.cuda.current_stream().wait_stream(s)
            torch.cuda.synchronize()
            runner, per = g.replay, graph_batch
            runner()
            torch.cuda.synchronize()
        except Exception:
            runner, per = fn, 1
    reps = max(1, iters // per)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        runner()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * per)


# ------------------------------------------------------------------ the CPU oracle as a baseline
def oracle_sample_c2(d, target_seconds=12.0):
    """Time the fp64 oracle on the first rows of the workload; returns (rows, seconds, cores)."""
    import oracle
    cores = oracle.get_threads()
    probe = 128
    t0 = time.perf_counter()
    oracle.gemm_epilogue(d["X"][:probe], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][:probe])
    dt = time.perf_counter() - t0
    rows = int(min(d["X"].shape[0], max(probe, (target_seconds / dt) * probe)))
    rows -= rows % 128
    t0 = time.perf_counter()
    oracle.gemm_epilogue(d["X"][:rows], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][:rows])
    return rows, time.perf_counter() - t0, cores


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    d = ki.gemm_inputs(WORKLOAD, seed=0)
    cores = oracle.get_threads()
    # size one step at ~6 s of CPU work so that warmup + steps end within a few minutes
    probe = 128
    t0 = time.perf_counter()
    oracle.gemm_epilogue(d["X"][:probe], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][:probe])
    dt = time.perf_counter() - t0
    per_step_s = 150.0 / max(1, args.steps + args.warmup)
    rows = int(min(M2, max(probe, (min(6.0, per_step_s) / dt) * probe)))
    rows -= rows % 128
    step = lambda: oracle.gemm_epilogue(d["X"][:rows], d["W"], d["b"], "gelu_tanh", 0.5, d["R"][:rows])
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    secs = time.perf_counter() - t0
    flops = 2.0 * rows * N2 * K2 * args.steps
    val = flops / secs / 1e12
    sample = "rows [0,%d) of X/R per step, all of W (%.3g of the workload's FLOPs)" % (rows, rows / M2)
    line = {
        "impl": "reference", "metric": "fused_chain_tflops", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": secs * 1e3 / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "c2: bf16 Linear+bias+GELU(tanh)*0.5+residual, X[8192,4096] W[4096,4096]",
                   "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ context: the other chains
def torch_unfused(name, t):
    """The same chain as separate eager torch ops (the paper's speedup denominator)."""
    import torch
    import torch.nn.functional as F
    if name == "c1":
        return lambda: torch.relu(F.linear(t["X"], t["W"], t["b"]))
    if name == "c2":
        return lambda: F.gelu(F.linear(t["X"], t["W"], t["b"]), approximate="tanh") * 0.5 + t["R"]
    if name == "c3":
        return lambda: torch.softmax(F.linear(t["X"], t["W"], t["b"]), dim=1)
    if name == "c4":
        return lambda: torch.sigmoid(F.linear(t["X"], t["W"], t["b"])).sum(dim=1, dtype=torch.float32)
    return lambda: F.group_norm(torch.relu(F.conv2d(t["x"], t["w"], t["bias"], padding=1)), 32, eps=1e-5)


def chain_table(kf, device, peaks, c2_tensors, c2_us):
    """us/call, TFLOP/s and roofline fractions of every benchmark chain + unfused torch."""
    import torch
    torch.backends.cuda.matmul.allow_tf32 = False
    torch.backends.cudnn.allow_tf32 = False
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)      # larger than the 126 MB L2
    c2_out = torch.empty(M2, N2, dtype=torch.bfloat16, device=device)
    specs = {
        "c1": dict(flops=2.0 * 128 * 256 * 512, bytes=4 * (128 * 512 + 256 * 512 + 256 + 128 * 256)),
        "c2": dict(flops=FLOPS_C2, bytes=ALG_BYTES_C2),
        "c3": dict(flops=2.0 * 4096 * 8192 * 2048, bytes=2 * (4096 * 2048 + 8192 * 2048 + 8192 + 4096 * 8192)),
        "c4": dict(flops=2.0 * 16384 * 1024 * 1024, bytes=2 * (16384 * 1024 + 1024 * 1024 + 1024) + 4 * 16384),
        "c5": dict(flops=2.0 * 128 * 64 * 64 * 128 * 576,
                   bytes=2 * (128 * 64 * 64 * 64 + 128 * 64 * 9 + 128 + 128 * 128 * 64 * 64)),
    }
    for name in ("c1", "c2", "c3", "c4", "c5"):
        if name == "c2":
            t = c2_tensors
        elif name == "c5":
            d = ki.conv_inputs("c5", seed=0)
            t = {k: to_dev(d[k], device) for k in ("x", "w", "bias")}
        else:
            d = ki.gemm_inputs(name, seed=0)
            t = {k: to_dev(d[k], device) for k in ("X", "W", "b")}
        if name == "c1":
            fn = lambda: kf.gemm_epilogue(t["X"], t["W"], t["b"], "relu")
        elif name == "c2":
            fn = None          # set below (needs t)
        elif name == "c3":
            o3 = torch.empty(4096, 8192, dtype=torch.bfloat16, device=device)
            fn = lambda: kf.gemm_rowreduce(t["X"], t["W"], t["b"], "none", "softmax", out=o3)
        elif name == "c4":
            o4 = torch.empty(16384, dtype=torch.float32, device=device)
            fn = lambda: kf.gemm_rowreduce(t["X"], t["W"], t["b"], "sigmoid", "sum", out=o4)
        else:
            o5 = torch.empty(128, 128, 64, 64, dtype=torch.bfloat16, device=device)
            fn = lambda: kf.conv3x3_epilogue(t["x"], t["w"], t["bias"], "relu", 32, 1e-5, out=o5)
        small = name in ("c1", "c4")
        if fn is None:
            fn = lambda: kf.gemm_epilogue(t["X"], t["W"], t["b"], "gelu_tanh", 0.5, t["R"], out=c2_out)
        n0 = kf.kf_launch_count()
        fn()
        kernels_per_call = int(kf.kf_launch_count() - n0)   # this library's kernels in one call: the route taken
        us = c2_us if name == "c2" else time_calls(fn, 200 if small else 40, 5, graph_batch=20 if small else 0)
        st = time_calls_stats(fn, 200 if small else 40, 5, graph_batch=20 if small else 0)
        us_torch = time_calls(torch_unfused(name, t), 200 if small else 20, 5, graph_batch=20 if small else 0)
        s = specs[name]
        tf = s["flops"] / us / 1e6
        gbs = s["bytes"] / us / 1e3
        # the roofline time of the chain: the slower of its FLOPs at the measured bf16 burst peak
        # (fp32 chain c1: launch-bound, reported for completeness) and its algorithmic bytes at the
        # measured HBM bandwidth
        t_roof = max(s["flops"] / (peaks["bf16_tflops"] * 1e6), s["bytes"] / (peaks["hbm_gbs"] * 1e3))
        out[name] = {
            "us_per_call": round(us, 3), "us_median": round(st["median"], 3), "us_min": round(st["min"], 3),
            "samples": st["samples"], "kernels_per_call": kernels_per_call, "tflops": round(tf, 2),
            "t_roof_us": round(t_roof, 3), "roofline_frac": round(t_roof / us, 4),
            "roofline_bound": "tensor" if s["flops"] / (peaks["bf16_tflops"] * 1e6) >= s["bytes"] / (peaks["hbm_gbs"] * 1e3) else "hbm",
            "frac_tensor_peak_measured_burst": round(tf / peaks["bf16_tflops"], 4),
            "frac_tensor_peak_nominal_2250": round(tf / 2250.0, 4),
            "algorithmic_gbs": round(gbs, 1), "frac_hbm_measured": round(gbs / peaks["hbm_gbs"], 4),
            "unfused_torch_us": round(us_torch, 3), "speedup_vs_unfused_torch": round(us_torch / us, 3),
        }
        if small:
            # these two fit in L2 (0.9 MB, 36 MB): the figures above are warm (back-to-back calls);
            # cold = a 256 MiB buffer is overwritten before every timed call
            cold = time_calls_stats(fn, 30, 3, flush=flush.zero_)
            out[name]["cache"] = "warm (L2-resident); cold variant beside it"
            out[name]["us_cold_median"] = round(cold["median"], 3)
            out[name]["us_cold_min"] = round(cold["min"], 3)
        if name == "c1":
            # launch-bound: the same call without CUDA-graph replay (host launch path included), and
            # an empty kernel launched the same two ways
            out[name]["us_per_call_eager"] = round(time_calls(fn, 400, 20), 3)
            out[name]["noop_kernel_us_graph"] = round(time_calls(kf.kf_launch_noop, 400, 20, graph_batch=20), 3)
            out[name]["noop_kernel_us_eager"] = round(time_calls(kf.kf_launch_noop, 400, 20), 3)
        del t
    # The paper's worked chain (Appendix C.2): matmul, add, swish, tanh, GELU(erf), hardtanh.  The
    # paper fuses only the five post-matmul operators (speedup 1.04 -> 1.31x on an RTX 5090);
    # here the whole chain is one kernel.  Shape: config 2's (the paper prints none).
    import torch.nn.functional as F
    t = c2_tensors
    oc = torch.empty(M2, N2, dtype=torch.bfloat16, device=device)
    n0 = kf.kf_launch_count()
    kf.gemm_epilogue(t["X"], t["W"], t["b"], "chain95", out=oc)
    k95 = int(kf.kf_launch_count() - n0)
    us = time_calls(lambda: kf.gemm_epilogue(t["X"], t["W"], t["b"], "chain95", out=oc), 40, 5)

    def torch_chain95():
        z = F.linear(t["X"], t["W"], t["b"])
        z = torch.sigmoid(z) * z
        z = torch.tanh(z)
        z = F.gelu(z)
        return F.hardtanh(z, -1.0, 1.0)

    us_torch = time_calls(torch_chain95, 20, 5)
    out["paper_chain_matmul_add_swish_tanh_gelu_hardtanh"] = {
        "shape": "config 2's X, W, b", "us_per_call": round(us, 3), "kernels_per_call": k95,
        "tflops": round(FLOPS_C2 / us / 1e6, 2), "unfused_torch_us": round(us_torch, 3),
        "speedup_vs_unfused_torch": round(us_torch / us, 3), "paper_speedup_rtx5090": 1.31}
    # The 2-D form of the paper's case-study chain (Appendix C.1): conv, softmax over channels,
    # two max-pools of 2 (= one of 4).  Shape: config 5's x, w, bias (the paper prints none).
    d = ki.conv_inputs("c5", seed=0)
    t5 = {k: to_dev(d[k], device) for k in ("x", "w", "bias")}
    op = torch.empty(128, 128, 16, 16, dtype=torch.bfloat16, device=device)
    n0 = kf.kf_launch_count()
    kf.conv3x3_softmax_pool(t5["x"], t5["w"], t5["bias"], 4, out=op)
    kpool = int(kf.kf_launch_count() - n0)
    us = time_calls(lambda: kf.conv3x3_softmax_pool(t5["x"], t5["w"], t5["bias"], 4, out=op), 40, 5)

    def torch_conv_softmax_pool():
        z = torch.softmax(F.conv2d(t5["x"], t5["w"], t5["bias"], padding=1), dim=1)
        return F.max_pool2d(F.max_pool2d(z, 2), 2)

    us_torch = time_calls(torch_conv_softmax_pool, 20, 5)
    out["paper_chain_conv_softmax_maxpool_maxpool_2d"] = {
        "shape": "config 5's x, w, bias; pool 2 twice", "us_per_call": round(us, 3), "kernels_per_call": kpool,
        "tflops": round(specs["c5"]["flops"] / us / 1e6, 2), "unfused_torch_us": round(us_torch, 3),
        "speedup_vs_unfused_torch": round(us_torch / us, 3)}
    return out


def run_single_workload(args, kf, device, peaks):
    """--workload cN: time one chain alone (used for profiling); prints a reduced JSON line."""
    import torch
    name = args.workload
    specs = {
        "c1": (2.0 * 128 * 256 * 512, 4 * (128 * 512 + 256 * 512 + 256 + 128 * 256)),
        "c3": (2.0 * 4096 * 8192 * 2048, 2 * (4096 * 2048 + 8192 * 2048 + 8192 + 4096 * 8192)),
        "c4": (2.0 * 16384 * 1024 * 1024, 2 * (16384 * 1024 + 1024 * 1024 + 1024) + 4 * 16384),
        "c5": (2.0 * 128 * 64 * 64 * 128 * 576, 2 * (128 * 64 * 64 * 64 + 128 * 64 * 9 + 128 + 128 * 128 * 64 * 64)),
    }
    specs["pool"] = (specs["c5"][0], 2 * (128 * 64 * 64 * 64 + 128 * 64 * 9 + 128 + 128 * 128 * 16 * 16))
    specs["f32"] = (2.0 * 2048 ** 3, 4 * (3 * 2048 * 2048 + 2048 + 2048 * 2048))
    specs["skinny"] = (2.0 * 64 * 8192 * 8192, 2 * (64 * 8192 + 8192 * 8192 + 8192 + 64 * 8192))
    flops, nbytes = specs[name]
    if name in ("f32", "skinny"):   # fp32 3xTF32 chain 2048^3; bf16 split-K cluster chain 64x8192x8192
        g = torch.Generator(device=device).manual_seed(0)
        dt = torch.float32 if name == "f32" else torch.bfloat16
        M, N, K = (2048, 2048, 2048) if name == "f32" else (64, 8192, 8192)
        X = torch.randn((M, K), generator=g, device=device).to(dt)
        W = (torch.randn((N, K), generator=g, device=device) * K ** -0.5).to(dt)
        b = torch.randn((N,), generator=g, device=device).to(dt)
        R = torch.randn((M, N), generator=g, device=device).to(dt)
        o = torch.empty((M, N), dtype=dt, device=device)
        fn = lambda: kf.gemm_epilogue(X, W, b, "gelu_tanh", 0.5, R, out=o)
    elif name == "pool":      # conv3x3 -> channel softmax -> max-pool 4 on config 5's tensors
        d = ki.conv_inputs("c5", seed=0)
        t = {k: to_dev(d[k], device) for k in ("x", "w", "bias")}
        o = torch.empty(128, 128, 16, 16, dtype=torch.bfloat16, device=device)
        fn = lambda: kf.conv3x3_softmax_pool(t["x"], t["w"], t["bias"], 4, out=o)
    elif name == "c5":
        d = ki.conv_inputs("c5", seed=0)
        t = {k: to_dev(d[k], device) for k in ("x", "w", "bias")}
        o = torch.empty(128, 128, 64, 64, dtype=torch.bfloat16, device=device)
        fn = lambda: kf.conv3x3_epilogue(t["x"], t["w"], t["bias"], "relu", 32, 1e-5, out=o)
    else:
        d = ki.gemm_inputs(name, seed=0)
        t = {k: to_dev(d[k], device) for k in ("X", "W", "b")}
        if name == "c1":
            fn = lambda: kf.gemm_epilogue(t["X"], t["W"], t["b"], "relu")
        elif name == "c3":
            o = torch.empty(4096, 8192, dtype=torch.bfloat16, device=device)
            fn = lambda: kf.gemm_rowreduce(t["X"], t["W"], t["b"], "none", "softmax", out=o)
        else:
            o = torch.empty(16384, dtype=torch.float32, device=device)
            fn = lambda: kf.gemm_rowreduce(t["X"], t["W"], t["b"], "sigmoid", "sum", out=o)
    l0 = kf.kf_launch_count()
    us = time_calls(fn, args.steps, max(3, args.warmup), graph_batch=0)
    tf = flops / us / 1e6
    print(json.dumps({"metric": "fused_chain_tflops", "value": round(tf, 3), "unit": "TFLOP/s",
                      "us_per_call": round(us, 3), "steps": args.steps, "warmup": max(3, args.warmup),
                      "algorithmic_gbs": round(nbytes / us / 1e3, 1),
                      "gpu_launches": int(kf.kf_launch_count() - l0),
                      "config": {"workload": name}, "data": "synthetic"}))


# ------------------------------------------------------------------ shape sweep (the paper's metrics)
# Synthetic shapes in the four categories of the paper's Table 2 (matmul-centered, mixed
# reduction, reduction-dominated, conv-centered); none is an item of the paper's benchmark suite.
SWEEP_GEMM = [  # (dtype, M, N, K, act, scale, residual)
    ("bf16", 128, 1024, 1024, "relu", 1.0, False), ("bf16", 512, 512, 512, "gelu_tanh", 1.0, False),
    ("bf16", 1024, 4096, 1024, "swish", 1.0, True), ("bf16", 2048, 2048, 2048, "gelu_erf", 0.5, True),
    ("bf16", 4096, 4096, 4096, "sigmoid", 1.0, False), ("bf16", 8192, 1024, 8192, "tanh", 2.0, False),
    ("bf16", 16384, 512, 512, "relu", 1.0, True), ("bf16", 1000, 1000, 1000, "gelu_tanh", 1.0, False),
    ("bf16", 4096, 11008, 4096, "swish", 1.0, False), ("bf16", 333, 777, 520, "hardtanh", 1.0, True),
    ("bf16", 8192, 4096, 4096, "chain95", 1.0, False), ("bf16", 64, 8192, 8192, "none", 1.0, False),
    ("f32", 128, 256, 512, "relu", 1.0, False), ("f32", 64, 64, 64, "gelu_tanh", 1.0, False),
    ("f32", 512, 512, 256, "sigmoid", 1.0, True),
    ("f32", 2048, 2048, 2048, "gelu_tanh", 1.0, True), ("f32", 1024, 4096, 1024, "relu", 1.0, False),
]
SWEEP_ROWRED = [  # (M, N, K, pre_act, red)
    (1024, 1024, 1024, "none", "softmax"), (4096, 8192, 2048, "none", "softmax"),
    (512, 32000, 1024, "none", "softmax"), (8192, 512, 512, "relu", "softmax"),
    (100, 1000, 304, "none", "softmax"),
    (16384, 1024, 1024, "sigmoid", "sum"), (4096, 4096, 1024, "gelu_tanh", "sum"),
    (1024, 512, 2048, "sigmoid", "sum"), (65536, 256, 256, "relu", "sum"),
]
SWEEP_CONV = [  # (Nb, Cin, H, W, Cout, groups [GroupNorm] or -pool [softmax + max-pool])
    (16, 64, 32, 32, 64, 8), (128, 64, 64, 64, 128, 32), (32, 128, 32, 32, 128, 16),
    (8, 64, 128, 128, 64, 4), (64, 64, 16, 16, 256, 32), (10, 3, 30, 30, 16, 4),
    (128, 64, 64, 64, 128, -4), (16, 64, 32, 32, 16, -2),
    (32, 64, 56, 56, 64, 8), (32, 128, 28, 28, 128, 8), (32, 256, 14, 14, 256, 8), (16, 3, 224, 224, 64, 8),
]
SWEEP_CONV_F32 = [(32, 64, 56, 56, 64, 8), (16, 64, 32, 32, 64, 8)]   # fp32, ReLU + GroupNorm
SWEEP_GEMM_GN = [(8192, 4096, 4096, 128), (1024, 1024, 1024, 32), (128, 1024, 512, 32)]   # bf16, GroupNorm + swish
SWEEP_CONV_GAP = [(128, 64, 64, 64, 128), (32, 64, 56, 56, 64)]        # bf16, ReLU + global average pool
SWEEP_CONV_POOL = [  # bf16 (Nb, Cin, H, W, Cout, act, kind, pool)
    (128, 64, 64, 64, 128, "relu", "max", 2), (128, 64, 64, 64, 128, "swish", "avg", 2),
    (32, 128, 32, 32, 128, "relu", "max", 2), (32, 64, 56, 56, 64, "relu", "max", 2),
    (16, 64, 128, 128, 64, "relu", "avg", 4),
]
SWEEP_ROWRED_F32 = [(2048, 4096, 1024, "none", "softmax"), (4096, 1024, 1024, "sigmoid", "sum")]


def _torch_act(name):
    import torch
    import torch.nn.functional as F
    return {"none": lambda z: z, "relu": torch.relu, "gelu_tanh": lambda z: F.gelu(z, approximate="tanh"),
            "gelu_erf": F.gelu, "sigmoid": torch.sigmoid, "swish": lambda z: torch.sigmoid(z) * z,
            "tanh": torch.tanh, "hardtanh": lambda z: F.hardtanh(z, -1.0, 1.0),
            "chain95": lambda z: F.hardtanh(F.gelu(torch.tanh(torch.sigmoid(z) * z)), -1.0, 1.0)}[name]


def run_sweep(kf, device):
    """Speedup of every sweep shape over the same chain as separate eager torch ops, and the
    paper's summary metrics (Section 4.1): fast_1 = share of shapes with speedup > 1, average
    and geometric-mean speedup.  Timing only; parity of these kernels is the tests' job."""
    import torch
    import torch.nn.functional as F
    torch.backends.cuda.matmul.allow_tf32 = False
    torch.backends.cudnn.allow_tf32 = False
    g = torch.Generator(device=device).manual_seed(0)
    rnd = lambda shape, dt, sc=1.0: (torch.randn(shape, generator=g, device=device) * sc).to(dt)
    rows = []

    def record(cat, name, fn, ref, flops):
        big = flops > 2e9
        us = time_calls(fn, 30 if big else 200, 5, graph_batch=0 if big else 20)
        ut = time_calls(ref, 20 if big else 200, 5, graph_batch=0 if big else 20)
        row = {"category": cat, "shape": name, "us": round(us, 2), "torch_us": round(ut, 2),
               "speedup": round(ut / us, 3), "tflops": round(flops / us / 1e6, 1)}
        if not big:
            # launch-bound shapes are replayed from CUDA graphs above; eager = plain calls in a loop,
            # host launch path (argument checks, dispatch, tensor-map lookup) included
            row["eager_us"] = round(time_calls(fn, 200, 10), 2)
            row["torch_eager_us"] = round(time_calls(ref, 200, 10), 2)
        rows.append(row)

    for dtn, M, N, K, act, scale, res in SWEEP_GEMM:
        dt = torch.bfloat16 if dtn == "bf16" else torch.float32
        X, W, b = rnd((M, K), dt), rnd((N, K), dt, K ** -0.5), rnd((N,), dt, K ** -0.5)
        R = rnd((M, N), dt) if res else None
        out = torch.empty((M, N), dtype=dt, device=device)
        ta = _torch_act(act)

        def ref(X=X, W=W, b=b, R=R, ta=ta, scale=scale):
            y = ta(F.linear(X, W, b))
            if scale != 1.0:
                y = y * scale
            return y + R if R is not None else y

        record("matmul-centered", "%s %dx%dx%d %s%s%s" % (dtn, M, N, K, act, "*s" if scale != 1.0 else "",
                                                           "+R" if res else ""),
               lambda X=X, W=W, b=b, R=R, out=out, act=act, scale=scale:
               kf.gemm_epilogue(X, W, b, act, scale, R, out=out), ref, 2.0 * M * N * K)
        del X, W, b, R, out
    for M, N, K, pre, red, dt in ([r + (torch.bfloat16,) for r in SWEEP_ROWRED] +
                                  [r + (torch.float32,) for r in SWEEP_ROWRED_F32]):
        X, W, b = rnd((M, K), dt), rnd((N, K), dt, K ** -0.5), rnd((N,), dt, K ** -0.5)
        ta = _torch_act(pre)
        if red == "softmax":
            out = torch.empty((M, N), dtype=dt, device=device)
            ref = lambda X=X, W=W, b=b, ta=ta: torch.softmax(ta(F.linear(X, W, b)), dim=1)
            cat = "mixed-reduction"
        else:
            out = torch.empty((M,), dtype=torch.float32, device=device)
            ref = lambda X=X, W=W, b=b, ta=ta: ta(F.linear(X, W, b)).sum(dim=1, dtype=torch.float32)
            cat = "reduction-dominated"
        record(cat, "%s %dx%dx%d %s->%s" % ("bf16" if dt == torch.bfloat16 else "f32", M, N, K, pre, red),
               lambda X=X, W=W, b=b, out=out, pre=pre, red=red: kf.gemm_rowreduce(X, W, b, pre, red, out=out),
               ref, 2.0 * M * N * K)
        del X, W, b, out
    for Nb, Cin, H, Wd, Cout, gp, dt in ([c + (torch.bfloat16,) for c in SWEEP_CONV] +
                                         [c + (torch.float32,) for c in SWEEP_CONV_F32]):
        dn = "bf16" if dt == torch.bfloat16 else "f32"
        x, w, b = rnd((Nb, Cin, H, Wd), dt), rnd((Cout, Cin, 3, 3), dt, (9 * Cin) ** -0.5), rnd((Cout,), dt, 0.1)
        flops = 2.0 * Nb * H * Wd * Cout * Cin * 9
        if gp > 0:
            out = torch.empty((Nb, Cout, H, Wd), dtype=dt, device=device)
            record("conv-centered", "%s conv %dx%dx%dx%d->%d relu GN%d" % (dn, Nb, Cin, H, Wd, Cout, gp),
                   lambda x=x, w=w, b=b, out=out, gp=gp: kf.conv3x3_epilogue(x, w, b, "relu", gp, 1e-5, out=out),
                   lambda x=x, w=w, b=b, gp=gp: F.group_norm(torch.relu(F.conv2d(x, w, b, padding=1)), gp, eps=1e-5),
                   flops)
        else:
            pool = -gp
            out = torch.empty((Nb, Cout, H // pool, Wd // pool), dtype=dt, device=device)
            record("conv-centered", "bf16 conv %dx%dx%dx%d->%d softmax pool%d" % (Nb, Cin, H, Wd, Cout, pool),
                   lambda x=x, w=w, b=b, out=out, pool=pool: kf.conv3x3_softmax_pool(x, w, b, pool, out=out),
                   lambda x=x, w=w, b=b, pool=pool: F.max_pool2d(torch.softmax(F.conv2d(x, w, b, padding=1), dim=1), pool),
                   flops)
        del x, w, b, out
    for M, N, K, groups in SWEEP_GEMM_GN:
        dt = torch.bfloat16
        X, W, b = rnd((M, K), dt), rnd((N, K), dt, K ** -0.5), rnd((N,), dt, K ** -0.5)
        ga, be = rnd((N,), dt, 0.1) + 1.0, rnd((N,), dt, 0.1)
        out = torch.empty((M, N), dtype=dt, device=device)

        def ref(X=X, W=W, b=b, ga=ga, be=be, groups=groups):
            z = F.group_norm(F.linear(X, W, b), groups, ga, be, 1e-5)
            return torch.sigmoid(z) * z

        record("mixed-reduction", "bf16 %dx%dx%d GroupNorm%d swish" % (M, N, K, groups),
               lambda X=X, W=W, b=b, ga=ga, be=be, out=out, groups=groups:
               kf.gemm_groupnorm(X, W, b, groups, 1e-5, ga, be, "swish", out=out), ref, 2.0 * M * N * K)
        del X, W, b, ga, be, out
    for Nb, Cin, H, Wd, Cout in SWEEP_CONV_GAP:
        dt = torch.bfloat16
        x, w, b = rnd((Nb, Cin, H, Wd), dt), rnd((Cout, Cin, 3, 3), dt, (9 * Cin) ** -0.5), rnd((Cout,), dt, 0.1)
        out = torch.empty((Nb, Cout), dtype=torch.float32, device=device)
        record("conv-centered", "bf16 conv %dx%dx%dx%d->%d relu global-avg-pool" % (Nb, Cin, H, Wd, Cout),
               lambda x=x, w=w, b=b, out=out: kf.conv3x3_act_gap(x, w, b, "relu", out=out),
               lambda x=x, w=w, b=b: torch.relu(F.conv2d(x, w, b, padding=1)).mean(dim=(2, 3)),
               2.0 * Nb * H * Wd * Cout * Cin * 9)
        del x, w, b, out
    for Nb, Cin, H, Wd, Cout, act, kind, pool in SWEEP_CONV_POOL:
        dt = torch.bfloat16
        x, w, b = rnd((Nb, Cin, H, Wd), dt), rnd((Cout, Cin, 3, 3), dt, (9 * Cin) ** -0.5), rnd((Cout,), dt, 0.1)
        out = torch.empty((Nb, Cout, H // pool, Wd // pool), dtype=dt, device=device)
        ta, tp = _torch_act(act), (F.max_pool2d if kind == "max" else F.avg_pool2d)
        record("conv-centered", "bf16 conv %dx%dx%dx%d->%d %s %s-pool%d" % (Nb, Cin, H, Wd, Cout, act, kind, pool),
               lambda x=x, w=w, b=b, out=out, act=act, kind=kind, pool=pool:
               kf.conv3x3_act_pool(x, w, b, act, kind, pool, out=out),
               lambda x=x, w=w, b=b, ta=ta, tp=tp, pool=pool: tp(ta(F.conv2d(x, w, b, padding=1)), pool),
               2.0 * Nb * H * Wd * Cout * Cin * 9)
        del x, w, b, out
    sp = np.array([r["speedup"] for r in rows])
    summary = {"shapes": len(rows), "fast_1": round(float((sp > 1.0).mean()), 3),
               "avg_speedup": round(float(sp.mean()), 3),
               "geomean_speedup": round(float(np.exp(np.log(sp).mean())), 3), "min_speedup": float(sp.min())}
    print(json.dumps({"metric": "speedup_over_unfused_torch", "summary": summary, "rows": rows,
                      "data": "synthetic", "config": {"workload": "sweep"}}))

# ------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the context table and baselines")
    ap.add_argument("--workload", default=WORKLOAD, choices=["c1", "c2", "c3", "c4", "c5", "pool", "f32", "skinny"],
                    help="c2 is the headline; the others print a reduced line (profiling aid); "
                         "pool = conv3x3 -> channel softmax -> max-pool on config 5's tensors; "
                         "f32 = fp32 2048^3 chain (3xTF32 kernel); skinny = bf16 64x8192x8192 (split-K)")
    ap.add_argument("--sweep", action="store_true",
                    help="time every sweep shape against unfused torch; prints fast_1 / avg / geomean")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the chains have no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    import paper_2605_30359_b200 as kf   # raises if libkf.so is missing
    kf.lib()
    peaks = load_peaks()
    if args.sweep:
        if rank == 0:
            run_sweep(kf, device)
        return
    if args.workload != WORKLOAD:
        if rank == 0:
            run_single_workload(args, kf, device, peaks)
        return

    # inputs: rank r works on its own batch (seed r); resident in HBM before the timed region
    d = ki.gemm_inputs(WORKLOAD, seed=rank_seed(rank))
    t = {k: to_dev(d[k], device) for k in ("X", "W", "b", "R")}
    Y = torch.empty(M2, N2, dtype=torch.bfloat16, device=device)
    step = lambda: kf.gemm_epilogue(t["X"], t["W"], t["b"], "gelu_tanh", 0.5, t["R"], out=Y)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = kf.kf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = kf.kf_launch_count() - launches0
    clocks = sampler.stop()
    if kf.kf_device_status() != kf.KF_OK:
        raise SystemExit("device status reports a timed-out wait: the run is invalid")
    ms = max_over_ranks(ms, world, device)
    ms_per_step = ms / args.steps
    value = whole_job_tflops(FLOPS_C2, world, ms_per_step)
    kernel_tflops = FLOPS_C2 / (ms_per_step * 1e-3) / 1e12          # one launch per step per rank

    # end to end: pinned host buffers in, host buffer out, copies inside the timed region
    hX, hW, hb, hR = (to_pinned(d[k]) for k in ("X", "W", "b", "R"))
    hY = torch.empty(M2, N2, dtype=torch.bfloat16).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        return kf.gemm_epilogue_host(hX, hW, hb, "gelu_tanh", 0.5, hR, out_host=hY, device=device)

    for _ in range(2):
        e2e_step()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms, world, device)
    e2e_val = whole_job_tflops(FLOPS_C2, world, e2e_ms / e2e_steps)
    h2d = sum(x.numel() * x.element_size() for x in (hX, hW, hb, hR))
    d2h = hY.numel() * hY.element_size()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    traffic = c2_traffic_bytes()
    line = {
        "metric": "fused_chain_tflops", "value": round(value, 2), "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(ms_per_step, 5), "us_per_call": round(ms_per_step * 1e3, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "c2: bf16 Linear+bias+GELU(tanh)*0.5+residual, X[8192,4096] W[4096,4096] "
                               "b[4096] R[8192,4096], fp32 accumulate, bf16 out",
                   "flops_per_step_per_gpu": FLOPS_C2, "l2": "inputs larger than L2 (235 MB per step)",
                   "parallelism": "replicas: each rank its own batch, no collective",
                   "peaks": peaks["_source"]},
        "clocks": clocks,
        "e2e": {"value": round(e2e_val, 2), "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "call": "kf_gemm_epilogue_host (C ABI, pinned host buffers, 4 row blocks)"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "umma_chain_kernel<256,elementwise,gelu_tanh>",
                     "achieved": round(kernel_tflops, 2), "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": round(kernel_tflops / peaks["bf16_tflops"], 4),
                     "frac_of_nominal_2250": round(kernel_tflops / 2250.0, 4),
                     "peak_source": peaks["_source"] + " cuBLAS bf16 burst",
                     "traffic": traffic,
                     "traffic_source": "ncu summary under profiles/ (one capture of this kernel)" if traffic else None},
    }
    if world == 1 and not args.no_extras:
        # a seconds-long leg of the same step, to set beside the sustained (power-capped) peak
        sus = ClockSampler(local)
        torch.cuda.synchronize()
        sus.start()
        n_sus, t0 = 0, time.perf_counter()
        e0.record()
        while time.perf_counter() - t0 < 2.2:
            for _ in range(50):
                step()
            n_sus += 50
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        sus_ms = e0.elapsed_time(e1)
        sus_clk = sus.stop()
        sus_tf = FLOPS_C2 * n_sus / (sus_ms * 1e-3) / 1e12
        line["sustained"] = {"seconds": round(sus_ms * 1e-3, 2), "steps": n_sus, "tflops": round(sus_tf, 2),
                             "us_per_call": round(sus_ms * 1e3 / n_sus, 2),
                             "peak_sustained": peaks["bf16_tflops_sustained"],
                             "frac_of_measured_sustained": round(sus_tf / peaks["bf16_tflops_sustained"], 4),
                             "sm_mhz_median": sus_clk["sm_mhz"], "reasons": sus_clk["reasons"],
                             "note": "includes a host synchronize every 50 steps"}
        rows, secs, cores = oracle_sample_c2(d)
        line["cpu_baseline"] = {
            "value": round(2.0 * rows * N2 * K2 / secs / 1e12, 6), "unit": "TFLOP/s", "cores": cores,
            "kind": "oracle", "seconds": round(secs, 2),
            "sample": "rows [0,%d) of X/R, all of W (%.3g of one step's FLOPs)" % (rows, rows / M2)}
        line["chains"] = chain_table(kf, device, peaks, t, ms_per_step * 1e3)
        line["paper_context"] = {"hardware": "RTX 5090", "matmul_centered_avg_speedup": 1.16,
                                 "conv_centered_avg_speedup": 1.33, "mixed_reduction_avg_speedup": 1.23,
                                 "reduction_dominated_avg_speedup": 6.56}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
