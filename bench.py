#!/usr/bin/env python
"""Benchmark of the Monarch hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one fused Monarch convolution (load, forward Monarch-DFT, spectrum multiply, inverse,
store) over the M2-BERT-base-shaped batch: x[32, 768, 512] bf16, circular, N = 512 = 32 x 16.
The step cycles through buffer sets that together exceed twice the L2 so DRAM traffic is real.
Prints ONE JSON line.  Multi-GPU: every rank runs the same per-GPU workload (rows are independent,
no collective on the data path); the value is the sum over ranks divided by the slowest rank's time.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "Monarch-conv tokens*channels/s"
UNIT = "tokens*ch/s"
WORKLOAD = "config2: bidirectional Monarch conv x[B=32,H=768,N=512] bf16, N=512=32x16, fp32 accumulate"
B2, H2, N2 = 32, 768, 512
L2_BYTES = 126 * 1024 * 1024
MIN_REGION_MS = 60.0   # shortest timed region: the K-step loop is repeated until it lasts this long
# DRAM bytes (read + write) of one launch of the dominant kernel from the ncu capture summarised in
# profiles/; None until a capture of the current kernel exists.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 28_521_472  # 28.37 MB read + 0.15 MB written inside the capture window (output still dirty in L2)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def reduce_max(value: float) -> float:
    """Max over ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        t = torch.tensor([value], dtype=torch.float64)
        if dist.get_backend() == "nccl":
            t = t.cuda()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return value


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


# ---- CPU baseline: the oracle as it stands, on a bounded sample ---------------------------------

def _oracle_rows(job):
    """Worker of the CPU-baseline pool: the oracle, as it stands, on a slice of channels (all batch rows of them)."""
    from oracle import monarch_oracle as O
    k64, x64, dims = job
    O.monarch_conv(k64[None], x64, dims, causal=False)
    return x64.shape[0] * x64.shape[1]


def oracle_conv_sample(reps: int = 8):
    """Times the oracle's Monarch conv on the full config-2 batch `reps` times, the channels split over a pool of one
    process per host core (the oracle itself is single-threaded numpy); returns (tokens*ch/s, processes used, description)."""
    import multiprocessing as mp
    from paper_2310_12109_b200 import synth
    c = synth.config2(B=B2, H=H2)
    k64, x64 = c["k"].astype(np.float64), c["x"].astype(np.float64)
    cores = max(1, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1))
    cores = min(cores, 64)
    per = -(-H2 // (4 * cores))                                 # ~4 slices per process
    jobs = [(k64[h0:h0 + per], np.ascontiguousarray(x64[:, h0:h0 + per]), c["dims"]) for h0 in range(0, H2, per)]
    ctx = mp.get_context("spawn")                               # no fork of a process that holds a CUDA context
    with ctx.Pool(cores) as pool:
        pool.map(_oracle_rows, jobs[:cores])                    # start-up and imports outside the timed region
        w0 = time.perf_counter()
        rows = 0
        for _ in range(reps):
            rows += sum(pool.map(_oracle_rows, jobs))
        wall = time.perf_counter() - w0
    assert rows == reps * B2 * H2
    return rows * N2 / wall, cores, (f"oracle.monarch_conv on the full config-2 batch ({B2 * H2} rows x {N2}), {reps} passes, channels split "
                                     f"over {cores} processes, {wall:.1f} s")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import monarch_oracle as O
    from paper_2310_12109_b200 import synth
    # each step: the oracle on a bounded sample of the same workload, sized so that the whole run
    # (warm-up + steps) stays near two minutes at the oracle's ~5e3 rows/s
    rows = int(5000 * 120.0 / max(1, args.steps + args.warmup))
    Bs = max(1, min(B2, rows // H2))
    Hs = H2 if rows >= H2 else max(8, rows)
    c = synth.config2(B=Bs, H=Hs)
    k64, x64 = c["k"].astype(np.float64)[None], c["x"].astype(np.float64)
    for _ in range(args.warmup):
        O.monarch_conv(k64, x64, c["dims"], causal=False)
    w0, c0 = time.perf_counter(), time.process_time()
    for _ in range(args.steps):
        O.monarch_conv(k64, x64, c["dims"], causal=False)
    wall, cpu = time.perf_counter() - w0, time.process_time() - c0
    value = args.steps * Bs * Hs * N2 / wall
    cores = max(1, int(round(cpu / wall)))
    sample = f"each step = oracle.monarch_conv on {Bs * Hs} of the {B2 * H2} rows (x {N2})"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * wall / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---- GPU arm ----------------------------------------------------------------------------------------

def time_launches(fn, n, torch):
    """CUDA-event time (ms) of n back-to-back calls of fn(i) on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def side_workloads(torch, M, synth, peaks, quick: bool, which=("config3", "config4", "config5", "operator", "backward", "hyena"), reps=None):
    """Config 3 (Monarch matmul), config 4 (order-3 causal conv) and config 5 (M2 block forward): time per call,
    throughput and roofline fraction, outside the headline timed region.  Configs 4 and 3 -- the other half of the metric --
    come last, so that a truncated copy of the line still ends with them."""
    out = {}
    reps = reps if reps is not None else (3 if quick else 10)
    bf = lambda a: torch.from_numpy(a).cuda().to(torch.bfloat16)  # noqa: E731
    if "hyena" in which:
        out.update(_side_hyena(torch, M, synth, peaks, reps, bf))
    if "backward" in which:
        out.update(_side_backward(torch, M, synth, peaks, reps, bf))
    if "operator" in which:
        out.update(_side_operator(torch, M, synth, peaks, reps, bf))
    if "config5" in which:
        out.update(_side_config5(torch, M, synth, peaks, reps, bf))
    if "config4" in which:
        out.update(_side_config4(torch, M, synth, peaks, max(reps, 10), bf))
    if "config3" in which:
        out.update(_side_config3(torch, M, synth, peaks, max(reps, 20), bf))
    return out


def _side_hyena(torch, M, synth, peaks, reps, bf):
    """The M2 Hyena layer with heads at B = 32, n = 256, d = 768, head dimension 16 (convolution plan N = 512): time per call."""
    B, n, d, dh = 32, 256, 768, 16
    torch.manual_seed(231012109)
    plan = M.Plan((32, 16), dtype=M.M2_BF16, device=torch.cuda.current_device())
    W = [(torch.randn(d, d, device="cuda") / d ** 0.5).to(torch.bfloat16) for _ in range(4)]
    kfs = [M.m2_kernel_spectrum(plan, torch.randn(d, n, device="cuda") * 0.05) for _ in range(3)]
    kfl = M.m2_kernel_spectrum(plan, torch.randn(d // dh, n, device="cuda") * 0.05)   # one long kernel per head
    u = torch.randn(B, n, d, device="cuda").to(torch.bfloat16)
    y = torch.empty_like(u)
    scratch = M.m2_hyena_scratch(plan, B, n, d, dh)
    f = lambda i: M.m2_hyena_heads_fwd(plan, u, W, kfs[0], kfs[1], kfs[2], kfl, dh, scratch=scratch, y=y)  # noqa: E731
    time_launches(f, 2, torch)
    ms = time_launches(f, reps, torch) / reps
    out = {"hyena_heads_layer": {"kernel": plan.last_kernel(), "ms": ms, "tokens_per_s": B * n / (ms * 1e-3),
                                 "shape": {"B": B, "n": n, "d": d, "head_dim": dh}, "scratch_MB": scratch.numel() / 1e6}}
    del scratch, kfl
    # the gated bidirectional M2-BERT sequence mixer at the M2-BERT-base shape (circular, n = N = 512)
    n = 512
    kf, kfr = (M.m2_kernel_spectrum(plan, torch.randn(d, n, device="cuda") * 0.05) for _ in range(2))
    ws = [torch.randn(d, 3, device="cuda") / 3 ** 0.5 for _ in range(3)]
    x = torch.randn(B, n, d, device="cuda").to(torch.bfloat16)
    y = torch.empty_like(x)
    scratch = torch.empty(int(M.lib().m2_bert_mixer_scratch_bytes(plan.handle, B, d)), dtype=torch.uint8, device="cuda")
    f = lambda i: M.m2_bert_mixer_fwd(plan, x, W, ws, kf, kfr, scratch=scratch, y=y)  # noqa: E731
    time_launches(f, 2, torch)
    ms = time_launches(f, reps, torch) / reps
    out["bert_gated_mixer"] = {"kernel": plan.last_kernel(), "ms": ms, "tokens_per_s": B * n / (ms * 1e-3), "shape": {"B": B, "n": n, "d": d},
                               "scratch_MB": scratch.numel() / 1e6}
    plan.close()
    return out


def _side_backward(torch, M, synth, peaks, reps, bf):
    """Gradient kernels on the config-2 and config-3 shapes: time per call (CUDA events), upstream gradients synthetic."""
    out = {}
    c = synth.config2(B=B2, H=H2)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=torch.cuda.current_device())
    kf = M.m2_kernel_spectrum(plan, torch.from_numpy(c["k"]).cuda())
    kfc = M.m2_spectrum_conjugate(plan, kf, H2)
    x = bf(c["x"])
    g = bf(synth.round_bf16(synth.normal(synth.stream_id(12, 0), c["x"].shape)))
    dx = torch.empty_like(x)
    ws = torch.empty(int(M.lib().m2_conv_bwd_workspace_bytes(plan.handle, B2, H2)), dtype=torch.uint8, device="cuda")
    f_dx = lambda i: M.m2_monarch_conv_fwd(plan, g, kfc, M.M2_CIRCULAR, y=dx)  # noqa: E731
    f_dk = lambda i: M.m2_monarch_conv_bwd_kernel(plan, x, g, M.M2_CIRCULAR, ws=ws)  # noqa: E731
    res = {}
    for name, f in (("dx", f_dx), ("dk", f_dk)):
        time_launches(f, 3, torch)
        res[name + "_ms"] = time_launches(f, reps, torch) / reps
        res[name + "_kernel"] = plan.last_kernel()
    out["config2_backward"] = res
    plan.close()
    del x, g, dx, ws
    B4, H4, n4 = 4, 1024, 16384
    c = synth.config4(B=B4, H=H4, n=n4)
    plan = M.Plan((32, 32, 32), dtype=M.M2_BF16, device=torch.cuda.current_device())
    x = bf(c["x"])
    g = bf(synth.round_bf16(synth.normal(synth.stream_id(12, 2), c["x"].shape)))
    ws = torch.empty(int(M.lib().m2_conv_bwd_workspace_bytes(plan.handle, B4, H4)), dtype=torch.uint8, device="cuda")
    f_dk = lambda i: M.m2_monarch_conv_bwd_kernel(plan, x, g, M.M2_CAUSAL, ws=ws)  # noqa: E731
    time_launches(f_dk, 2, torch)
    out["config4_backward"] = {"dk_ms": time_launches(f_dk, reps, torch) / reps, "dk_kernel": plan.last_kernel(),
                               "note": "dx = the forward kernel with the conjugated spectrum (same time as the forward pass)"}
    plan.close()
    del x, g, ws
    T, b = 16384, 64
    c = synth.config3(T=T, b=b)
    plan = M.Plan((b, b), dtype=M.M2_BF16, device=torch.cuda.current_device())
    L, R, X = bf(c["L"]), bf(c["R"]), bf(c["X"])
    G = bf(synth.round_bf16(synth.normal(synth.stream_id(12, 1), c["X"].shape)))
    ws = torch.empty(int(M.lib().m2_matmul_bwd_workspace_bytes(plan.handle, T)), dtype=torch.uint8, device="cuda")
    f_dX = lambda i: M.m2_monarch_matmul_bwd_input(plan, G, L, R, ws=ws)  # noqa: E731
    f_dW = lambda i: M.m2_monarch_matmul_bwd_weights(plan, X, G, L, R, ws=ws)  # noqa: E731
    res = {}
    for name, f in (("dX", f_dX), ("dL_dR", f_dW)):
        time_launches(f, 3, torch)
        res[name + "_ms"] = time_launches(f, reps, torch) / reps
        res[name + "_kernel"] = plan.last_kernel()
    out["config3_backward"] = res
    plan.close()
    return out


def _side_operator(torch, M, synth, peaks, reps, bf):
    """The paper's operator benchmark (Table 2): M_b (K (.) M_a X) with learnable order-2 Monarch matrices, block size
    sqrt(N), X in R^{N x 768} with the columns as the vectors (m2_monarch_cols, two calls); FLOP utilisation =
    8 N sqrt(N) flops per column / time / the measured bf16 burst peak.  Random-normal device data (timing only)."""
    out = {}
    d = 768
    paper = {4096: (4.78, 11.1), 16384: (12.7, 32.1), 65536: (25.6, 41.4), 262144: (42.8, 53.7)}
    torch.manual_seed(231012109)
    for b in (64, 128, 256, 512):
        N = b * b
        plan = M.Plan((b, b), dtype=M.M2_BF16, device=torch.cuda.current_device())
        W = [(torch.randn(b, b, b, device="cuda") / b ** 0.5).to(torch.bfloat16) for _ in range(4)]
        X = torch.randn(1, N, d, device="cuda").to(torch.bfloat16)
        K = torch.randn(N, d, device="cuda").to(torch.bfloat16)
        Y1, Y2, ws = torch.empty_like(X), torch.empty_like(X), torch.empty_like(X)

        def f(i):
            M.m2_monarch_cols(plan, X, W[0], W[1], K, M.M2_ACT_NONE, Y=Y1, ws=ws)
            M.m2_monarch_cols(plan, Y1, W[2], W[3], None, M.M2_ACT_NONE, Y=Y2, ws=ws)
        time_launches(f, 3, torch)
        r = max(reps, 20) if b <= 128 else max(reps, 5)
        ms = time_launches(f, r, torch) / r
        ms_graph = None
        if b <= 128:   # the four launches are host-bound at these sizes: also time them replayed from a CUDA graph
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                f(0)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=st):
                    for _ in range(10):
                        f(0)
                g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(st)
                for _ in range(10):
                    g.replay()
                e1.record(st)
            torch.cuda.synchronize()
            ms_graph = e0.elapsed_time(e1) / 100
        fl = 8.0 * N * b * d
        by = 4 * (2 * N * d * 2 + b * b * b * 2) + N * d * 2   # per stage: rows in, rows out, one factor; + the kernel K once
        t_roof = max(fl / (peaks["bf16_tflops_sustained"] * 1e12), by / (peaks["hbm_gbs"] * 1e9))
        out[f"operator_N{N}"] = {
            "kernel": plan.last_kernel(), "ms": ms, "TFLOPs": fl / (ms * 1e9), "launches_per_call": 4,
            "flop_utilisation_pct": 100 * fl / (ms * 1e9) / peaks["bf16_tflops"], "roofline_frac": t_roof / (ms * 1e-3),
            "paper_flop_utilisation_pct": {"A100": paper[N][0], "RTX4090": paper[N][1]}}
        if ms_graph is not None:
            out[f"operator_N{N}"].update({"ms_cuda_graph": ms_graph, "flop_utilisation_pct_cuda_graph": 100 * fl / (ms_graph * 1e9) / peaks["bf16_tflops"]})
        plan.close()
        del W, X, K, Y1, Y2, ws
    # the same operator at N = 4096 with the vectors as rows (tokens contiguous in N): m2_monarch_mix
    N, b, T = 4096, 64, 768
    plan = M.Plan((b, b), dtype=M.M2_BF16, device=torch.cuda.current_device())
    W = [(torch.randn(b, b, b, device="cuda") / 8.0).to(torch.bfloat16) for _ in range(4)]
    K = torch.randn(T, N, device="cuda").to(torch.bfloat16)
    X = torch.randn(T, N, device="cuda").to(torch.bfloat16)
    Y = torch.empty_like(X)
    ws = M.m2_matmul_workspace(plan, T)
    f = lambda i: M.m2_monarch_mix(plan, X, K, W[0], W[1], W[2], W[3], act=M.M2_ACT_NONE, Y=Y, ws=ws)  # noqa: E731
    time_launches(f, 3, torch)
    r = max(reps, 20)
    ms = time_launches(f, r, torch) / r
    fl = 8.0 * T * N * b
    out["operator_N4096_rows"] = {"kernel": plan.last_kernel(), "ms": ms, "TFLOPs": fl / (ms * 1e9), "launches_per_call": 4,
                                  "flop_utilisation_pct": 100 * fl / (ms * 1e9) / peaks["bf16_tflops"]}
    plan.close()
    return out


def _side_config3(torch, M, synth, peaks, reps, bf):
    out = {}
    T, b = 16384, 64
    c = synth.config3(T=T, b=b)
    plan = M.Plan((b, b), dtype=M.M2_BF16, device=torch.cuda.current_device())
    L, R = bf(c["L"]), bf(c["R"])
    Xs = [bf(c["X"]) for _ in range(2)]
    Ys = [torch.empty_like(Xs[0]) for _ in range(2)]
    ws = M.m2_matmul_workspace(plan, T)
    f = lambda i: M.m2_monarch_matmul(plan, Xs[i % 2], L, R, Ys[i % 2], ws=ws)  # noqa: E731
    time_launches(f, 3, torch)
    ms = time_launches(f, reps, torch) / reps
    by = 2 * T * b * b * 2 + 2 * b * b * b * 2   # x read + y write + both weight sets (the workspace round trip is not algorithmic)
    fl = 4.0 * T * b * b * b
    out["config3_matmul"] = {
        "kernel": plan.last_kernel(), "ms": ms, "elements_per_s": T * b * b / (ms * 1e-3), "algorithmic_GBps": by / (ms * 1e6),
        "TFLOPs": fl / (ms * 1e9), "roofline": {"bound": "hbm", "achieved": by / (ms * 1e6), "peak": peaks["hbm_gbs"],
                                                 "unit": "GB/s", "frac": by / (ms * 1e6) / peaks["hbm_gbs"]}}
    plan.close()
    return out


def _side_config4(torch, M, synth, peaks, reps, bf):
    out = {}
    B, H, n = 4, 1024, 16384
    c = synth.config4(B=B, H=H, n=n)
    plan = M.Plan((32, 32, 32), dtype=M.M2_BF16, device=torch.cuda.current_device())
    kf = M.m2_kernel_spectrum(plan, torch.from_numpy(c["k"]).cuda())
    xs = [bf(c["x"]) for _ in range(2)]
    ys = [torch.empty_like(xs[0]) for _ in range(2)]
    f = lambda i: M.m2_monarch_conv_fwd(plan, xs[i % 2], kf, M.M2_CAUSAL, y=ys[i % 2])  # noqa: E731
    time_launches(f, 2, torch)
    ms = time_launches(f, reps, torch) / reps
    by = 2 * B * H * n * 2 + H * 32768 * 8               # x + y (bf16) + fp32 spectrum (the format in use)
    fl_plain = 2.0 * (2 + 4 + 4) * 32768 * 32 * 2 * B * H   # plain count: real first stage, complex after, fwd + inv, nothing skipped
    # the variant implemented: two real rows ride as one complex row (every stage complex, 8 N 32 flops, half as many rows); the
    # zero half of the first digit is skipped on the way in (half of the first stage's K steps) and not produced on the way out
    # (half of the last stage's columns): 6 stages -> 0.5 + 4 + 0.5 = 5 stage-equivalents per pair
    fl = 2.0 * 4 * 32768 * 32 * (0.5 + 1 + 1 + 1 + 1 + 0.5) * (B * H / 2)
    t_hbm = by / (peaks["hbm_gbs"] * 1e9)
    t_tc = fl / (peaks["bf16_tflops_sustained"] * 1e12)
    bound = "tensor" if t_tc > t_hbm else "hbm"
    ach = fl / (ms * 1e9) if bound == "tensor" else by / (ms * 1e6)
    pk = peaks["bf16_tflops_sustained"] if bound == "tensor" else peaks["hbm_gbs"]
    out["config4_conv_order3"] = {
        "kernel": plan.last_kernel(), "ms": ms, "tokens_ch_per_s": B * H * n / (ms * 1e-3), "algorithmic_GBps": by / (ms * 1e6),
        "TFLOPs_executed": fl / (ms * 1e9), "TFLOPs_plain_count": fl_plain / (ms * 1e9),
        "frac_of_plain_count_tensor_roof": fl_plain / (ms * 1e9) / peaks["bf16_tflops_sustained"],
        "note": "roofline against the variant implemented (row pairs packed as complex rows, zero half of the first digit skipped: "
                f"{fl / 1e9:.1f} GFLOP executed, {by / 1e6:.1f} MB with the fp32 spectrum); the plain count is kept as a side key",
        "roofline": {"bound": bound, "achieved": ach, "peak": pk, "unit": "TFLOP/s" if bound == "tensor" else "GB/s", "frac": ach / pk}}
    plan.close()
    return out


def _side_config5(torch, M, synth, peaks, reps, bf):
    """M2 block forward [32, 512, 768]: sequence mix + gate + block-diagonal MLP (3 launches: transpose, gated conv, MLP)."""
    out = {}
    B, T, C = 32, 512, 768
    c = synth.config5(B=B, T=T, C=C)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=torch.cuda.current_device())
    kf = M.m2_kernel_spectrum(plan, torch.from_numpy(c["k"]).cuda())
    xs = [bf(c["x"]) for _ in range(3)]
    w = torch.from_numpy(c["w_short"]).cuda()
    Wu, Wd = bf(c["W_up"]), bf(c["W_down"])
    f = lambda i: M.m2_block_fwd(plan, xs[i % 3], kf, w, Wu, Wd)  # noqa: E731
    time_launches(f, 3, torch)
    ms = time_launches(f, reps, torch) / reps
    fl = 2.0 * 2 * B * T * C * (4 * C // 4)               # the MLP's two block-diagonal GEMMs (38.65 GFLOP)
    by = 2 * B * T * C * 2 + 2 * Wu.numel() * 2 + C * T * 8   # x in, y out, weights, spectrum
    t_tc = fl / (peaks["bf16_tflops_sustained"] * 1e12)
    out["config5_block"] = {
        "kernel": plan.last_kernel(), "ms": ms, "tokens_ch_per_s": B * T * C / (ms * 1e-3), "mlp_TFLOPs_if_all_time_were_mlp": fl / (ms * 1e9),
        "note": "whole block (transpose, conv with the gate in its last hand-off, MLP); roofline = the MLP's tensor time plus the conv's HBM time",
        "roofline": {"bound": "tensor", "achieved": fl / (ms * 1e9), "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": (t_tc + by / (peaks["hbm_gbs"] * 1e9)) / (ms * 1e-3)}}
    plan.close()
    return out


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2310_12109_b200 import binding as M
    from paper_2310_12109_b200 import build as BLD
    from paper_2310_12109_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group(backend="nccl", init_method="env://")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    BLD.build()
    peaks = measured_peaks()

    c = synth.config2(B=B2, H=H2)
    plan = M.Plan(c["dims"], dtype=M.M2_BF16, device=local_rank)
    kf = M.m2_kernel_spectrum(plan, torch.from_numpy(c["k"]).cuda())
    x0 = torch.from_numpy(c["x"]).cuda().to(torch.bfloat16)
    set_bytes = 2 * x0.numel() * 2 + B2 * 0 + H2 * N2 * 8
    nsets = max(2, -(-2 * L2_BYTES // set_bytes))          # rotate through > 2 x L2
    xs = [x0] + [x0.clone() for _ in range(nsets - 1)]
    ys = [torch.empty_like(x0) for _ in range(nsets)]

    def step(i):
        M.m2_monarch_conv_fwd(plan, xs[i % nsets], kf, M.M2_CIRCULAR, y=ys[i % nsets])

    warm = max(args.warmup, 3)
    for i in range(warm):
        step(i)
    torch.cuda.synchronize()
    # The step is tens of microseconds and successive launches overlap (programmatic dependent launch), so a timed region of
    # K steps can be far too short to measure: the K-step loop is repeated until the region lasts at least MIN_REGION_MS and
    # the time is reported per step.  The repeat count comes from an untimed estimate and is agreed on by all ranks.
    est = time_launches(step, max(args.steps, 20), torch) / max(args.steps, 20)
    rounds = int(reduce_max(float(max(1, -(-MIN_REGION_MS // max(est * args.steps, 1e-6))))))
    sampler = ClockSampler(local_rank)
    launches0 = plan.launch_count()
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(rounds):
        for i in range(args.steps):
            step(i)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    ms_total = reduce_max(e0.elapsed_time(e1))
    launches = plan.launch_count() - launches0      # kernels launched inside the timed region
    timed_steps = rounds * args.steps
    # keep the GPU under the same load a little longer if the timed region was too short to sample
    if sampler.nv is not None and len(sampler.samples) < 5:
        t_end = time.perf_counter() + 0.25
        i = 0
        while time.perf_counter() < t_end:
            step(i)
            i += 1
        torch.cuda.synchronize()
    clocks = sampler.stop()
    kernel_name = plan.last_kernel()
    ms_step = ms_total / timed_steps
    units = B2 * H2 * N2
    value = world * units / (ms_step * 1e-3)
    alg_bytes = 2 * units * 2 + H2 * N2 * 8                 # x read + y write (bf16) + the spectrum once
    achieved = alg_bytes / (ms_step * 1e6)                  # GB/s

    # end to end through the host-buffer entry point: pinned host x -> device -> conv -> host y, every step.
    # Two streams (each with its own plan, device scratch and pinned result buffer) alternate, so one step's
    # device->host copy runs while the next step's host->device copy does: PCIe is full duplex.
    xh = x0.cpu().pin_memory()
    yhs = [torch.empty_like(xh).pin_memory() for _ in range(2)]
    plans2 = [plan, M.Plan(c["dims"], dtype=M.M2_BF16, device=local_rank)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    e2e_steps = max(4, min(args.steps, 20))

    def e2e_step(i):
        with torch.cuda.stream(streams[i % 2]):
            M.m2_monarch_conv_fwd_host(plans2[i % 2], xh, kf, yhs[i % 2], xs[i % 2], ys[i % 2], M.M2_CIRCULAR)

    for i in range(4):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(streams[0])
    streams[1].wait_event(e0)
    for i in range(e2e_steps):
        e2e_step(i)
    streams[0].wait_stream(streams[1])
    e1.record(streams[0])
    torch.cuda.synchronize()
    ms_e2e = reduce_max(e0.elapsed_time(e1)) / e2e_steps
    plans2[1].close()
    e2e_value = world * units / (ms_e2e * 1e-3)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
        "timed_steps": timed_steps, "timed_region_ms": ms_total, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": f"rotates {nsets} buffer sets of {set_bytes / 1e6:.1f} MB (> 2 x L2)",
                   "kernel": kernel_name, "parallelism": f"dp{world} (independent rows, no collective)"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": units * 2, "d2h_bytes_per_step": units * 2,
                "ms_per_step": ms_e2e, "pipeline": "2 streams, double-buffered"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                     "peak_source": peaks["source"], "algorithmic_bytes_per_launch": alg_bytes},
    }
    plan.close()
    if rank == 0 and world == 1:
        if not args.no_cpu:
            v, cores, sample = oracle_conv_sample()
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
        if not args.no_side:
            del xs, ys
            torch.cuda.empty_cache()
            w = side_workloads(torch, M, synth, peaks, quick=args.quick)
            line["workloads"] = w
            # the other kernels the metric names, lifted to short keys at the end of the line
            if "config4_conv_order3" in w:
                line["roofline_conv3"] = dict(w["config4_conv_order3"]["roofline"], ms=w["config4_conv_order3"]["ms"], workload="config4")
            if "config3_matmul" in w:
                line["roofline_matmul"] = dict(w["config3_matmul"]["roofline"], ms=w["config3_matmul"]["ms"], workload="config3")
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-baseline leg")
    ap.add_argument("--no-side", action="store_true", help="skip the config-3 / config-4 side measurements")
    ap.add_argument("--quick", action="store_true", help="fewer repetitions of the side measurements")
    ap.add_argument("--only", default=None, choices=["config3", "config4", "config5", "operator", "backward", "hyena"],
                    help="run just this side workload (--steps launches after 2 warm-ups) and print its JSON; used for profiling")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.only:
        import torch
        from paper_2310_12109_b200 import binding as M
        from paper_2310_12109_b200 import build as BLD
        from paper_2310_12109_b200 import synth
        BLD.build()
        torch.cuda.set_device(0)
        print(json.dumps(side_workloads(torch, M, synth, measured_peaks(), True, which=(args.only,), reps=max(1, args.steps))))
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: become the launcher (one rank per GPU, as torchrun would start them)
        sys.exit(launch_ranks(args))
    else:
        world = int(os.environ.get("WORLD_SIZE", "1"))
        if world != args.gpus:
            sys.stderr.write(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}; start it with --nproc-per-node {args.gpus}\n")
            sys.exit(2)
        run_gpu(args)


def launch_ranks(args) -> int:
    """`python bench.py --gpus N` with N > 1 and no launcher: re-runs this command under torch.distributed.run with N ranks on
    this node (127.0.0.1 rendezvous).  Refuses (exit 2) when the node has fewer than N GPUs."""
    import subprocess
    import torch
    have = torch.cuda.device_count()
    if have < args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} asked for, {have} CUDA device(s) visible\n")
        return 2
    port = 29500 + (os.getpid() % 2000)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


if __name__ == "__main__":
    main()
