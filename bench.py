#!/usr/bin/env python
"""Benchmark of the SQ-format hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic activations of the
70B-decoder-shaped prefill linears (M = 4096 tokens through the fused-QKV, O, fused gate-up
and down projections; b = 128, k = 16 static positions): for each linear, sq_encode of its
bf16 input followed by sq_gemm against its packed INT4 weights.  `value` is the effective
throughput 2*M*N*K summed over the four linears divided by the step time (encode included),
with inputs resident in HBM; `e2e` is the same metric with the inputs in pinned host memory
and the outputs copied back inside the timed region.  The roofline object covers the GEMM
kernel (tensor bound); `encode` reports the bandwidth-bound encode kernel on the 8192 x 8192
bandwidth test.  `--impl reference` times the CPU oracle on a bounded sample instead.
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

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "sq_gemm effective TOPS (% of INT8 tensor peak); sq_encode GB/s (% of HBM)"
UNIT = "TOPS"
WORKLOAD = "70B-decoder-shaped prefill linears: M=4096 x (K,N) in {(8192,10240),(8192,8192),(8192,57344),(28672,8192)}; b=128,k=16 static"
SHAPES_70B = [(8192, 10240), (8192, 8192), (8192, 57344), (28672, 8192)]
SHAPES_8B = [(4096, 6144), (4096, 4096), (4096, 28672), (14336, 4096)]
M_70B, BANK_70B, K_70B = 4096, 128, 16
INT8_OVER_BF16 = 2.0        # nominal dense INT8 : bf16 tensor rate on B200 (4.5 : 2.25 PFLOP/s)
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
# ncu DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one gemm_kernel launch on the
# small capture case of profiles/gemm_kernel_static_b128_k16_M2048_N8192_K8192.txt, and that case's
# algorithmic bytes; the benchmark's launches are too large to capture with --set full, so their
# traffic is this ratio times their own algorithmic bytes (the traffic is operand streaming and
# grows with the operands).  It is below 1 because most of the output is still in L2 at kernel end.
GEMM_CAPTURE_TRAFFIC_BYTES = 50.89e6 + 4.22e6
GEMM_CAPTURE_ALGO_BYTES = 2048 * 8192 * 0.625 + 8192 * 8192 * 0.625 + 2.0 * 2048 * 8192
# ncu DRAM traffic of one encode launch of the 8192 x 8192 bandwidth test (dynamic k=8 / static k=8),
# profiles/encode_kernels_b64_k8_8192x8192.txt
ENCODE_TRAFFIC_BYTES_PER_LAUNCH = {"dynamic": 134.29e6 + 25.98e6, "static": 134.34e6 + 20.21e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, flag in zip(names, parts[2:6]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


# ----------------------------------------------------------------------------- the CUDA arm

class Linear:
    """One linear layer of the workload: packed weights, static positions, I/O buffers."""

    def __init__(self, sq, M, K, N, bank, k, static, seed, dev, dist="student_t3", independent_scales=False,
                 fused_a8=False):
        self.M, self.K, self.N = M, K, N
        self.fmt = sq.make_format(bank, k, static, independent_scales=independent_scales)
        W = gen.weights(N, K, seed=seed, device=dev)
        self.pos = None
        if static:
            calib = gen.calibration_batch(512, K, seed=seed, dist=dist, outlier_fraction=0.01,
                                          outlier_scale=20.0, device=dev)
            self.pos = sq.sq_calib_positions(sq.make_format(bank, k, True), calib, W)
            del calib
        self.w = sq.sq_pack_weights(self.fmt, W, self.pos)
        del W
        self.X = gen.activations(M, K, seed=seed, dist=dist, outlier_fraction=0.01, outlier_scale=20.0, device=dev)
        self.enc = sq.alloc_encoded(self.fmt, M, K, dev)
        self.out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        self.ops = 2.0 * M * N * K
        # algorithmic bytes: packed activations + packed weights + bf16 output
        payload = 0.5 + (1.0 if static else 2.0) * k / bank
        self.gemm_bytes = M * K * payload + N * K * (0.5 + (k / bank if static else 0.0)) + 2.0 * M * N
        self.encode_bytes = M * K * (2.0 + payload) + 9.0 * M
        # producer fusion: sq_encode_a8 writes the product's merged 8-bit operand next to the codes
        # (one more byte per element written by the encode, none of the expansion pass's traffic)
        self.fused_a8 = fused_a8 and static and not independent_scales and M > 128
        self.a8 = None
        if self.fused_a8:
            self.a8 = torch.empty(M, K, dtype=torch.uint8, device=dev)
            self.encode_bytes += float(M) * K
        self.launches = 2 if self.fused_a8 else 2 + (1 if sq.sq_gemm_workspace_bytes(self.fmt, M, N, K) else 0)

    def step(self, sq, events=None):
        if events is not None:
            events[0].record()
        if self.fused_a8:
            sq.sq_encode_a8(self.fmt, self.X, self.pos, out=self.enc, a8=self.a8)
        else:
            sq.sq_encode(self.fmt, self.X, self.pos, out=self.enc)
        if events is not None:
            events[1].record()
        if self.fused_a8:
            sq.sq_gemm_a8(self.fmt, self.enc, self.a8, self.w, self.pos, out=self.out)
        else:
            sq.sq_gemm(self.fmt, self.enc, self.w, self.pos, out=self.out)
        if events is not None:
            events[2].record()


def time_launches(fn, iters, warmup):
    """Median and best CUDA-event time (ms) of fn(i) over `iters` launches after `warmup`."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for i in range(iters):
        evs[i][0].record()
        fn(i)
        evs[i][1].record()
    torch.cuda.synchronize()
    times = [a.elapsed_time(b) for a, b in evs]
    return statistics.median(times), min(times)


def bench_encode_only(sq, dev, peaks, iters=50, warmup=10):
    """The bandwidth test: 8192 x 8192 bf16, Student-t with 0.5% channels x50, b=64, k in {4,8,16}.
    Next to every point: a plain device copy (torch) that moves the same number of bytes, timed the
    same way in the same run -- what a launch of this size can reach at all on this GPU."""
    M = K = 8192
    rows = []
    # three input buffers in rotation (384 MB > L2) so no launch finds its input in L2
    Xs = [gen.activations(M, K, seed=s, outlier_fraction=0.005, outlier_scale=50.0, device=dev) for s in range(3)]
    calib = gen.calibration_batch(512, K, seed=0, outlier_fraction=0.005, outlier_scale=50.0, device=dev)
    copy_dst = torch.empty(M * K, dtype=torch.bfloat16, device=dev)
    for static in (False, True):
        for k in (4, 8, 16):
            fmt = sq.make_format(64, k, static)
            pos = sq.sq_calib_positions(fmt, calib) if static else None
            enc = sq.alloc_encoded(fmt, M, K, dev)
            ms, best = time_launches(lambda i: sq.sq_encode(fmt, Xs[i % 3], pos, out=enc), iters, warmup)
            nbytes = M * K * (2.0 + 0.5 + (1.0 if static else 2.0) * k / 64) + 9.0 * M
            gbs = nbytes / (ms * 1e-3) / 1e9
            n_copy = int(nbytes / 4)          # bf16 elements: read + write = nbytes
            cms, _ = time_launches(lambda i: copy_dst[:n_copy].copy_(Xs[i % 3].view(-1)[:n_copy]), iters, warmup)
            copy_gbs = nbytes / (cms * 1e-3) / 1e9
            rows.append(["static" if static else "dynamic", k, round(ms * 1e3, 1), round(best * 1e3, 1), round(gbs),
                         round(gbs / peaks["hbm_gbs"], 3), round(gbs / 8000.0, 3), round(copy_gbs), round(gbs / copy_gbs, 3)])
    # sq_decode of the same tensor (k = 8): packed codes in, bf16 out; three encodings in rotation
    dec_rows = []
    out = torch.empty(M, K, dtype=torch.bfloat16, device=dev)
    for static in (False, True):
        fmt = sq.make_format(64, 8, static)
        pos = sq.sq_calib_positions(fmt, calib) if static else None
        encs = [sq.sq_encode(fmt, Xs[i], pos) for i in range(3)]
        ms, best = time_launches(lambda i: sq.sq_decode(fmt, encs[i % 3], pos, out=out), iters, warmup)
        nbytes = M * K * (2.0 + 0.5 + (1.0 if static else 2.0) * 8 / 64) + 8.0 * M
        gbs = nbytes / (ms * 1e-3) / 1e9
        dec_rows.append(["static" if static else "dynamic", 8, round(ms * 1e3, 1), round(best * 1e3, 1), round(gbs),
                         round(gbs / peaks["hbm_gbs"], 3)])
        del encs
    return {"cols": ["positions", "k", "us_median", "us_best", "GBps", "of_measured_hbm", "of_8TBps",
                     "same_run_copy_GBps", "of_same_run_copy"],
            "rows": rows, "launches": iters,
            "traffic_ncu_bytes_per_launch_k8": ENCODE_TRAFFIC_BYTES_PER_LAUNCH,
            "decode": {"cols": ["positions", "k", "us_median", "us_best", "GBps", "of_measured_hbm"], "rows": dec_rows}}


def graph_replay_us(fn, calls=10, replays=5):
    """GPU time per call of fn() when `calls` of them are replayed from a CUDA graph (no host cost)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        fn()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(calls):
                fn()
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(replays):
        graph.replay()
    g1.record()
    torch.cuda.synchronize()
    us = g0.elapsed_time(g1) * 1e3 / (calls * replays)
    del graph
    return us


def bench_8b_dynamic(sq, dev, peaks, iters=20):
    """sq_encode + sq_gemm on the 8B-decoder-shaped linears with dynamic positions (b=64, k=8) at
    M in {1, 16, 128, 2048}, plus the single-GEMM configuration (M=64, K=N=4096, N(0,1) activations).
    M >= 128: TOPS of the call the binding makes (with its workspace) and of plain sq_gemm (sparse
    part merged inside the GEMM kernel).  M <= 128: also the GPU time per call replayed from a CUDA
    graph and the INT4 weight stream N*K/2 bytes over it (those calls are host-bound otherwise)."""
    rows = []
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    shapes = [(K, N, M, "student_t3") for (K, N) in SHAPES_8B for M in (1, 16, 128, 2048)] + [(4096, 4096, 64, "normal")]
    for (K, N, M, dist) in shapes:
        l = Linear(sq, M, K, N, 64, 8, False, seed=K + N + M, dev=dev, dist=dist)
        e_ms, _ = time_launches(lambda i: sq.sq_encode(l.fmt, l.X, l.pos, out=l.enc), iters, 5)
        g_ms, _ = time_launches(lambda i: sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out), iters, 10)
        f_ms, _ = time_launches(lambda i: sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out, use_workspace=False), iters, 5)
        tops, ftops = l.ops / (g_ms * 1e-3) / 1e12, l.ops / (f_ms * 1e-3) / 1e12
        graph_us = wgbs = enc_graph_us = pair_graph_us = norm_pair_graph_us = None
        if M <= 128:
            graph_us = round(graph_replay_us(lambda: sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out)), 1)
            wgbs = round(N * K / 2 / (graph_us * 1e-6) / 1e9)
            enc_graph_us = round(graph_replay_us(lambda: sq.sq_encode(l.fmt, l.X, l.pos, out=l.enc)), 1)

            def pair():  # the product may fetch its first weight tiles while the encode still runs
                sq.sq_encode(l.fmt, l.X, l.pos, out=l.enc)
                sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out)
            pair_graph_us = round(graph_replay_us(pair), 1)
            gamma = torch.ones(K, dtype=torch.bfloat16, device=dev)

            def norm_pair():  # the same chain with the layer normalisation inside the encode
                sq.sq_rmsnorm_encode(l.fmt, l.X, gamma, 1e-5, None, out=l.enc, want_a8=False)
                sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out)
            try:
                norm_pair_graph_us = round(graph_replay_us(norm_pair), 1)
            except sq.SqError:
                norm_pair_graph_us = None
        rows.append([M, K, N, round(e_ms * 1e3, 1), round(g_ms * 1e3, 1), graph_us, wgbs, round(tops, 1),
                     round(tops / int8_peak, 3), round(tops / 4500.0, 3), round(f_ms * 1e3, 1), round(ftops, 1), enc_graph_us,
                     pair_graph_us, norm_pair_graph_us])
        del l
        torch.cuda.empty_cache()
    return {"cols": ["M", "K", "N", "encode_us", "gemm_us", "gemm_us_graph_replay", "weight_stream_GBps_graph_replay",
                     "TOPS", "of_measured_int8", "of_nominal_4500", "fused_gemm_us", "fused_TOPS", "encode_us_graph_replay",
                     "encode_plus_gemm_us_graph_replay", "rmsnorm_encode_plus_gemm_us_graph_replay"],
            "rows": rows}


def bench_decode_static(sq, dev, peaks):
    """Few tokens with STATIC positions (b=64, k=8) on the 8B-decoder shapes: GPU time per call of sq_gemm
    and of the chain sq_encode -> sq_gemm replayed from a CUDA graph, and the INT4 weight stream over the
    product's time."""
    rows = []
    fmt = sq.make_format(64, 8, True)
    for (K, N) in SHAPES_8B:
        W = gen.weights(N, K, seed=K + N, device=dev)
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(512, K, seed=K, outlier_fraction=0.01, outlier_scale=20.0, device=dev), W)
        w = sq.sq_pack_weights(fmt, W, pos)
        del W
        for M in (1, 16):
            X = gen.activations(M, K, seed=M, outlier_fraction=0.01, outlier_scale=20.0, device=dev)
            enc = sq.sq_encode(fmt, X, pos)
            out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
            g_us = graph_replay_us(lambda: sq.sq_gemm(fmt, enc, w, pos, out=out))

            def pair():
                sq.sq_encode(fmt, X, pos, out=enc)
                sq.sq_gemm(fmt, enc, w, pos, out=out)
            p_us = graph_replay_us(pair)
            gbs = N * K / 2 / (g_us * 1e-6) / 1e9
            rows.append([M, K, N, round(g_us, 1), round(gbs), round(gbs / peaks["hbm_gbs"], 3), round(p_us, 1)])
        del w
        torch.cuda.empty_cache()
    return {"cols": ["M", "K", "N", "gemm_us_graph_replay", "weight_stream_GBps", "of_measured_hbm", "encode_plus_gemm_us_graph_replay"],
            "rows": rows}


def bench_gemm_fused(sq, layers, dev, peaks, iters=10):
    """Plain sq_gemm (no workspace): the sparse INT8 part runs inside the GEMM kernel -- static
    positions as TMA-fed gathered K steps, dynamic positions merged into the widened activation
    tile -- against the call with a workspace (activations expanded once into 8-bit operands by a
    kernel of their own), on the 70B-shaped linears of the step (static, M = 4096) and, with
    dynamic positions b=128 k=16, on the same shapes."""
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    rows = []
    for l in layers:
        for ws in (False, True):
            ms, _ = time_launches(lambda i: sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out, use_workspace=ws), iters, 3)
            tops = l.ops / (ms * 1e-3) / 1e12
            rows.append([l.K, l.N, l.M, "static", "workspace" if ws else "fused", round(ms * 1e3, 1), round(tops, 1),
                         round(tops / int8_peak, 3), round(tops / 4500.0, 3)])
    for (K, N) in SHAPES_70B[:2]:
        l = Linear(sq, M_70B, K, N, BANK_70B, K_70B, False, seed=K + N, dev=dev)
        sq.sq_encode(l.fmt, l.X, l.pos, out=l.enc)
        for ws in (False, True):
            ms, _ = time_launches(lambda i: sq.sq_gemm(l.fmt, l.enc, l.w, l.pos, out=l.out, use_workspace=ws), iters, 3)
            tops = l.ops / (ms * 1e-3) / 1e12
            rows.append([K, N, l.M, "dynamic", "workspace" if ws else "fused", round(ms * 1e3, 1), round(tops, 1),
                         round(tops / int8_peak, 3), round(tops / 4500.0, 3)])
        del l
        torch.cuda.empty_cache()
    return {"cols": ["K", "N", "M", "positions", "mode", "gemm_us", "TOPS", "of_measured_int8", "of_nominal_4500"],
            "rows": rows}


def bench_weights_sq(sq, dev, peaks):
    """Weights in SQ-format (Algorithm 1's format, b=64, k=8 INT8 values per bank) against per-token INT8
    activations on the 8B-decoder shapes at 1 and 4 tokens: GPU time per call replayed from a CUDA graph
    and the weight stream (0.5 + k/b bytes per weight) over it."""
    rows = []
    fmt = sq.make_format(64, 8, True)
    for (K, N) in SHAPES_8B:
        W = gen.weights(N, K, seed=K + N, device=dev)
        enc = sq.sq_w_encode(fmt, W, (W.float() ** 2).contiguous())
        del W
        for M in (1, 4):
            xq, s_x = sq.sq_w_act_quant(gen.activations(M, K, seed=M, outlier_fraction=0.01, outlier_scale=20.0, device=dev))
            out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
            us = graph_replay_us(lambda: sq.sq_w_gemm(fmt, xq, s_x, enc, out=out))
            gbs = N * K * (0.5 + 8 / 64) / (us * 1e-6) / 1e9
            rows.append([M, K, N, round(us, 1), round(gbs), round(gbs / peaks["hbm_gbs"], 3)])
        del enc
        torch.cuda.empty_cache()
    return {"cols": ["M", "K", "N", "gemm_us_graph_replay", "weight_stream_GBps", "of_measured_hbm"], "rows": rows}


def bench_producer_fusion(sq, dev, peaks, iters=30):
    """sq_rmsnorm_encode (the normalisation that produces two of a decoder layer's four activations, computed
    inside the static-position encode) next to sq_encode of an already normalised tensor and to a library
    normalisation (torch rms_norm: read + write of the bf16 tensor, yardstick only): the fused call saves the
    normalised tensor's trip to memory and back.  Three inputs in rotation (> L2)."""
    rows = []
    for M, K, b, k in ((8192, 8192, 64, 8), (4096, 8192, 128, 16), (8192, 4096, 64, 8)):
        fmt = sq.make_format(b, k, True)
        Xs = [gen.activations(M, K, seed=s, outlier_fraction=0.005, outlier_scale=50.0, device=dev) for s in range(3)]
        gamma = (1.0 + 0.1 * gen.weights(1, K, seed=1, std=1.0, device=dev).float()).to(torch.bfloat16).reshape(K).contiguous()
        pos = sq.sq_calib_positions(fmt, gen.calibration_batch(512, K, seed=0, outlier_fraction=0.005, outlier_scale=50.0, device=dev), None)
        enc = sq.alloc_encoded(fmt, M, K, dev)
        a8 = torch.empty(M, K, dtype=torch.uint8, device=dev)
        t_e, _ = time_launches(lambda i: sq.sq_encode(fmt, Xs[i % 3], pos, out=enc), iters, 5)
        t_e8, _ = time_launches(lambda i: sq.sq_encode_a8(fmt, Xs[i % 3], pos, out=enc, a8=a8), iters, 5)
        t_f, _ = time_launches(lambda i: sq.sq_rmsnorm_encode(fmt, Xs[i % 3], gamma, 1e-5, pos, out=enc, want_a8=False), iters, 5)
        t_f8, _ = time_launches(lambda i: sq.sq_rmsnorm_encode(fmt, Xs[i % 3], gamma, 1e-5, pos, out=enc, a8=a8), iters, 5)
        try:
            t_n, _ = time_launches(lambda i: torch.nn.functional.rms_norm(Xs[i % 3], (K,), gamma, 1e-5), 10, 3)
        except Exception:
            t_n = None
        nbytes = M * K * (2.0 + 0.5 + k / b)
        rows.append([M, K, b, k, round(t_f * 1e3, 1), round(nbytes / (t_f * 1e-3) / 1e9), round(nbytes / (t_f * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
                     round(t_f8 * 1e3, 1), round(t_e * 1e3, 1), round(t_e8 * 1e3, 1), None if t_n is None else round(t_n * 1e3, 1)])
        del Xs, enc, a8
        torch.cuda.empty_cache()
    return {"cols": ["M", "K", "b", "k", "rmsnorm_encode_us", "GBps", "of_measured_hbm", "rmsnorm_encode_a8_us", "encode_us",
                     "encode_a8_us", "library_rms_norm_us"], "rows": rows}


def bench_layer_prefill(sq, layers, dev, iters=10):
    """The benchmark step's four linears as they sit in a decoder layer: the first (fused QKV) and the third
    (fused gate-up) read the output of a root-mean-square normalisation.  One pass = 4 x (encode + product)
    with (a) that normalisation inside the encode (sq_rmsnorm_encode), (b) a library normalisation
    (torch rms_norm, yardstick only) before sq_encode_a8, (c) no normalisation at all (the step `value` is
    quoted on).  Attention and the gated activation are not part of any of the three."""
    normed = [l for l in layers[0::2] if l.fused_a8]
    if len(normed) != 2 or len(layers) != 4:
        return None
    gam = {id(l): (1.0 + 0.1 * gen.weights(1, l.K, seed=7, std=1.0, device=dev).float()).to(torch.bfloat16).reshape(l.K).contiguous()
           for l in normed}
    try:
        sq.sq_rmsnorm_encode(normed[0].fmt, normed[0].X, gam[id(normed[0])], 1e-5, normed[0].pos, out=normed[0].enc, a8=normed[0].a8)
    except sq.SqError:
        return None

    def one_pass(mode):
        for l in layers:
            if id(l) in gam and mode == "fused":
                sq.sq_rmsnorm_encode(l.fmt, l.X, gam[id(l)], 1e-5, l.pos, out=l.enc, a8=l.a8)
            elif id(l) in gam and mode == "library":
                y = torch.nn.functional.rms_norm(l.X, (l.K,), gam[id(l)], 1e-5)
                sq.sq_encode_a8(l.fmt, y, l.pos, out=l.enc, a8=l.a8)
            else:
                sq.sq_encode_a8(l.fmt, l.X, l.pos, out=l.enc, a8=l.a8)
            sq.sq_gemm_a8(l.fmt, l.enc, l.a8, l.w, l.pos, out=l.out)
    # the three variants take turns, so that a drift of the clocks under the power cap hits them alike
    modes = ("fused", "library", "none")
    try:
        for mode in modes:
            one_pass(mode)
        torch.cuda.synchronize()
        evs = {mode: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)] for mode in modes}
        for i in range(iters):
            for mode in modes:
                evs[mode][i][0].record()
                one_pass(mode)
                evs[mode][i][1].record()
        torch.cuda.synchronize()
        res = {mode: round(statistics.median(a.elapsed_time(b) for a, b in evs[mode]), 4) for mode in modes}
    except Exception:
        return None
    ops = sum(l.ops for l in layers)
    return {"ms_norm_inside_encode": res["fused"], "ms_library_norm_then_encode": res["library"], "ms_no_norm": res["none"],
            "TOPS_norm_inside_encode": None if res["fused"] is None else round(ops / (res["fused"] * 1e-3) / 1e12, 1)}


def bench_same_run_int8(dev, iters=10):
    """A vendor INT8 GEMM (torch._int_mm, M=4096, N=K=8192) timed in the same run: a yardstick for
    the tensor pipe's INT8 rate at this run's clocks, never on the product path."""
    M, K, N = 4096, 8192, 8192
    try:
        a = torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev)
        b = torch.randint(-7, 8, (N, K), dtype=torch.int8, device=dev).t()
        ms, _ = time_launches(lambda i: torch._int_mm(a, b), iters, 3)
        return 2.0 * M * N * K / (ms * 1e-3) / 1e12
    except Exception:
        return None


def bench_int8_tensor_rate(sq):
    """The library's tensor-rate probe (tcgen05.mma.kind::i8 on shared-memory-resident operands and
    nothing else, one CTA per SM) timed in the same run: the INT8 rate the tensor pipe itself
    sustains -- for ~5 ms (boost clocks) and for a quarter of a second (under the power cap)."""
    def once(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ops = sq.sq_probe_int8_tensor_rate(iters)
        b.record()
        torch.cuda.synchronize()
        return ops / (a.elapsed_time(b) * 1e-3) / 1e12
    once(2000)
    burst = statistics.median(once(20000) for _ in range(5))
    sustained = once(1000000)

    def once_fp8(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ops = sq.sq_probe_fp8_tensor_rate(iters)
        b.record()
        torch.cuda.synchronize()
        return ops / (a.elapsed_time(b) * 1e-3) / 1e12
    once_fp8(2000)
    fp8_burst = statistics.median(once_fp8(20000) for _ in range(5))
    return burst, sustained, fp8_burst


def bench_format_sweep(sq, dev, peaks, iters=5):
    """The format-parameter sweep at M = 4096, K = N = 8192: bank b in {32, 64, 128} x high-precision
    fraction k/b in {1/16, 1/8, 1/4}, dynamic positions, static positions and static positions with
    independent scales of the two parts, outlier channels x10 and x50.
    Per point: sq_gemm time (median of CUDA-event pairs, pre-widened mode) and the relative
    Frobenius error of the bf16 output against the fp32 product of the bf16 inputs (a library
    matmul, used only as the yardstick)."""
    M, K, N = 4096, 8192, 8192
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    tf32 = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    res, fp_enc = [], []
    W = gen.weights(N, K, seed=5, device=dev)
    for scale in (10.0, 50.0):
        X = gen.activations(M, K, seed=5, outlier_fraction=0.01, outlier_scale=scale, device=dev)
        calib = gen.calibration_batch(512, K, seed=5, outlier_fraction=0.01, outlier_scale=scale, device=dev)
        ref = X.float() @ W.float().t()
        ref_norm = float(ref.norm())
        out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        for b in (32, 64, 128):
            for frac in (16, 8, 4):
                k = b // frac
                for static, indep in ((False, False), (True, False), (True, True)):
                    fmt = sq.make_format(b, k, static, independent_scales=indep)
                    pos = sq.sq_calib_positions(sq.make_format(b, k, True), calib, W) if static else None
                    w = sq.sq_pack_weights(fmt, W, pos)
                    enc = sq.sq_encode(fmt, X, pos)
                    for _ in range(3):
                        sq.sq_gemm(fmt, enc, w, pos, out=out)
                    torch.cuda.synchronize()
                    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
                    for e0, e1 in evs:
                        e0.record()
                        sq.sq_gemm(fmt, enc, w, pos, out=out)
                        e1.record()
                    torch.cuda.synchronize()
                    ms = statistics.median(a.elapsed_time(c) for a, c in evs)
                    tops = 2.0 * M * N * K / (ms * 1e-3) / 1e12
                    err = float((out.float() - ref).norm()) / ref_norm
                    res.append([b, k, ("indep" if indep else "static") if static else "dynamic", int(scale),
                                round(ms * 1e3, 1), round(tops), round(tops / int8_peak, 3), round(err, 4)])
                    del w, enc
                # floating-point variant (sparse FP8 E4M3 + dense FP4 E2M1 activations, FP4 weights): the same
                # shape on the FP8 tensor path (nominal rate = the INT8 one, so the same denominator)
                for static in (False, True):
                    fmt = sq.make_format(b, k, static)
                    pos = sq.sq_calib_positions(fmt, calib, W) if static else None
                    wf = sq.sq_fp_pack_weights(W)
                    encf, a8 = sq.sq_fp_encode(fmt, X, pos)
                    ms, _ = time_launches(lambda i: sq.sq_fp_gemm(encf, a8, wf, out=out), iters, 3)
                    tops = 2.0 * M * N * K / (ms * 1e-3) / 1e12
                    err = float((out.float() - ref).norm()) / ref_norm
                    res.append([b, k, "fp8/fp4 static" if static else "fp8/fp4 dynamic", int(scale), round(ms * 1e3, 1),
                                round(tops), round(tops / int8_peak, 3), round(err, 4)])
                    if b == 64 and k == 8 and scale == 10.0:
                        ems, _ = time_launches(lambda i: sq.sq_fp_encode(fmt, X, pos, out=encf, a8=a8), iters, 2)
                        nbytes = M * K * (2.0 + 0.5 + (1.0 if static else 2.0) * k / b + 1.0)
                        fp_enc.append(["static" if static else "dynamic", round(ems * 1e3, 1),
                                       round(nbytes / (ems * 1e-3) / 1e9)])
                    del wf, encf, a8
        del X, calib, ref, out
        torch.cuda.empty_cache()
    torch.backends.cuda.matmul.allow_tf32 = tf32
    return {"cols": ["b", "k", "positions", "outlier_scale", "gemm_us", "TOPS", "of_measured_int8", "rel_err_vs_fp32"],
            "rows": res,
            # sq_fp_encode at this shape, b=64, k=8 (codes, sparse entries and the merged 8-bit operand written)
            "fp_encode": {"cols": ["positions", "us", "GBps"], "rows": fp_enc}}


def oracle_sample(K, N, bank, k, seed, rows=32, cols=512):
    """Times the CPU oracle (encode + GEMM) on a bounded sample of one linear of the workload."""
    import oracle
    Xb = gen.bf16_bits(gen.activations(rows, K, seed=seed, outlier_fraction=0.01, outlier_scale=20.0))
    Wb = gen.bf16_bits(gen.weights(cols, K, seed=seed))
    calib = gen.bf16_bits(gen.calibration_batch(64, K, seed=seed, outlier_fraction=0.01, outlier_scale=20.0))
    pos = oracle.calib_positions(bank, k, calib, Wb)
    pw = oracle.pack_weights(bank, k, Wb, pos)
    t0 = time.perf_counter()
    enc = oracle.encode(bank, k, Xb, pos)
    oracle.gemm(bank, k, enc, pw, pos)
    dt = time.perf_counter() - t0
    return 2.0 * rows * cols * K, dt, oracle.num_threads()


def run_reference(args):
    """CPU oracle arm: same metric and config, each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    K, N = SHAPES_70B[1]
    sample = {"rows": 256, "cols": 2048}
    for _ in range(args.warmup):
        oracle_sample(K, N, BANK_70B, K_70B, 0, **sample)
    ops = dt = 0.0
    cores = 1
    for _ in range(args.steps):
        o, d, cores = oracle_sample(K, N, BANK_70B, K_70B, 0, **sample)
        ops += o
        dt += d
    tops = ops / dt / 1e12
    desc = f"encode + GEMM of {sample['rows']} token rows x {sample['cols']} output channels of the (K,N)=({K},{N}) linear per step"
    line = {"impl": "reference", "metric": METRIC, "value": tops, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
            "cpu_baseline": {"value": tops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": tops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


PROFILE_CASES = ("encode_dynamic", "encode_static", "encode_static_a8", "encode_rmsnorm", "encode_rmsnorm_a8", "gemm_a8", "gemm_stream",
                 "fp_gemm", "wsq_gemm")


def run_profile_case(args):
    """A handful of launches of one kernel on a small case, and nothing else: the command a profiler
    capture is taken of (inputs larger than L2 where the kernel streams from memory, well under
    1 GB on the device).  Prints one line naming the case; it is not a benchmark."""
    import paper_2512_05409_b200 as sq
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    case, n = args.profile_case, 6
    if case.startswith("encode"):
        M = K = 8192
        static = case != "encode_dynamic"
        fmt = sq.make_format(64, 8, static)
        Xs = [gen.activations(M, K, seed=s, outlier_fraction=0.005, outlier_scale=50.0, device=dev) for s in range(3)]
        pos = None
        if static:
            calib = gen.calibration_batch(512, K, seed=0, outlier_fraction=0.005, outlier_scale=50.0, device=dev)
            pos = sq.sq_calib_positions(fmt, calib, None)
        enc = sq.alloc_encoded(fmt, M, K, dev)
        a8 = torch.empty(M, K, dtype=torch.uint8, device=dev) if case.endswith("_a8") else None
        gamma = torch.ones(K, dtype=torch.bfloat16, device=dev)
        for i in range(n):
            if case.startswith("encode_rmsnorm"):
                sq.sq_rmsnorm_encode(fmt, Xs[i % 3], gamma, 1e-5, pos, out=enc, a8=a8, want_a8=a8 is not None)
            elif a8 is not None:
                sq.sq_encode_a8(fmt, Xs[i % 3], pos, out=enc, a8=a8)
            else:
                sq.sq_encode(fmt, Xs[i % 3], pos, out=enc)
    elif case == "gemm_a8":
        l = Linear(sq, 2048, 8192, 8192, BANK_70B, K_70B, True, seed=1, dev=dev, fused_a8=True)
        for _ in range(n):
            l.step(sq)
    elif case == "gemm_stream":
        K, N = SHAPES_8B[2]
        l = Linear(sq, 16, K, N, 64, 8, False, seed=2, dev=dev)
        for _ in range(n):
            l.step(sq)
    elif case == "fp_gemm":
        M, K, N = 2048, 8192, 8192
        fmt = sq.make_format(64, 8, False)
        W = gen.weights(N, K, seed=3, device=dev)
        w = sq.sq_fp_pack_weights(W)
        enc, a8 = sq.sq_fp_encode(fmt, gen.activations(M, K, seed=3, device=dev))
        out = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        for _ in range(n):
            sq.sq_fp_gemm(enc, a8, w, out=out)
    elif case == "wsq_gemm":
        K, N = SHAPES_8B[2]
        fmt = sq.make_format(64, 8, True)
        W = gen.weights(N, K, seed=4, device=dev)
        enc = sq.sq_w_encode(fmt, W, (W.float() ** 2).contiguous())
        xq, s_x = sq.sq_w_act_quant(gen.activations(4, K, seed=4, device=dev))
        out = torch.empty(4, N, dtype=torch.bfloat16, device=dev)
        for _ in range(n):
            sq.sq_w_gemm(fmt, xq, s_x, enc, out=out)
    torch.cuda.synchronize()
    assert sq.sq_device_status() == sq.SQ_OK
    print(json.dumps({"profile_case": case, "launches": n}))


def run_cuda(args):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    import paper_2512_05409_b200 as sq
    peaks = load_peaks()

    # weak scaling: every rank owns its own batch of M tokens (tokens are independent units)
    M = args.m
    chosen = [int(x) for x in args.linears.split(",")] if args.linears else list(range(len(SHAPES_70B)))
    layers = [Linear(sq, M, SHAPES_70B[i][0], SHAPES_70B[i][1], BANK_70B, K_70B, True, seed=rank * 16 + i, dev=dev,
                     independent_scales=args.independent_scales, fused_a8=not args.separate_expand)
              for i in chosen]
    total_ops = sum(l.ops for l in layers)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        for l in layers:
            l.step(sq)
    barrier()
    assert sq.sq_device_status() == sq.SQ_OK

    # ---- device-resident timing (inputs larger than L2: ~0.9 GB of packed weights + activations per step)
    evs = [[[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in layers] for _ in range(args.steps)]
    with ClockSampler(physical_gpu_index(local)) as clocks:
        barrier()
        t_first = torch.cuda.Event(enable_timing=True)
        t_last = torch.cuda.Event(enable_timing=True)
        t_first.record()
        for s in range(args.steps):
            for li, l in enumerate(layers):
                l.step(sq, evs[s][li])
        t_last.record()
        barrier()
        total_ms = t_first.elapsed_time(t_last)
        if total_ms < 1500:      # keep the sampler alive long enough to see the loaded clocks
            t_end = time.time() + 1.0
            while time.time() < t_end:
                for l in layers:
                    l.step(sq)
                torch.cuda.synchronize()
    clk = clocks.summary()
    assert sq.sq_device_status() == sq.SQ_OK

    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms_max = float(t.item())
    ms_per_step = total_ms_max / args.steps
    value = world * total_ops / (ms_per_step * 1e-3) / 1e12

    gemm_ms = sum(e[1].elapsed_time(e[2]) for st in evs for e in st)
    enc_ms = sum(e[0].elapsed_time(e[1]) for st in evs for e in st)
    n_gemm = args.steps * len(layers)
    gemm_tops = total_ops * args.steps / (gemm_ms * 1e-3) / 1e12
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    enc_bytes = sum(l.encode_bytes for l in layers) * args.steps
    enc_gbs = enc_bytes / (enc_ms * 1e-3) / 1e9

    # ---- end to end: pinned host inputs, device->host outputs, all inside the timed region
    host_X = [torch.empty(l.X.shape, dtype=torch.bfloat16).pin_memory() for l in layers]
    host_out = [torch.empty(l.out.shape, dtype=torch.bfloat16).pin_memory() for l in layers]
    for hx, l in zip(host_X, layers):
        hx.copy_(l.X)
    h2d = sum(hx.numel() * 2 for hx in host_X)
    d2h = sum(ho.numel() * 2 for ho in host_out)
    e2e_steps = max(1, min(args.steps, 3))

    # Three streams: host->device copies, compute, device->host copies.  A linear's input buffer is
    # refilled only after the previous step's kernels have read it, and its output buffer is
    # overwritten only after the previous step's copy-out has left it.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in layers]
    ev_done = [torch.cuda.Event() for _ in layers]
    ev_out = [torch.cuda.Event() for _ in layers]
    first = [True]

    def e2e_step():
        for i, (hx, ho, l) in enumerate(zip(host_X, host_out, layers)):
            with torch.cuda.stream(s_in):
                if not first[0]:
                    s_in.wait_event(ev_done[i])
                l.X.copy_(hx, non_blocking=True)
                ev_in[i].record(s_in)
            cur.wait_event(ev_in[i])
            if not first[0]:
                cur.wait_event(ev_out[i])
            l.step(sq)
            ev_done[i].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                ho.copy_(l.out, non_blocking=True)
                ev_out[i].record(s_out)
        first[0] = False

    s_in.wait_stream(cur)
    s_out.wait_stream(cur)
    e2e_step()
    cur.wait_stream(s_out)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    cur.wait_stream(s_in)
    cur.wait_stream(s_out)
    e1.record()
    barrier()
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_value = world * total_ops / (float(t.item()) / e2e_steps * 1e-3) / 1e12

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": (WORKLOAD if not args.linears else WORKLOAD + f" [subset {args.linears}]")
                               + (" [variant: independent scales of the two parts]" if args.independent_scales else ""), "M_per_gpu": M, "bank": BANK_70B, "k": K_70B, "positions": "static",
                   "step": ("sq_encode_a8 + sq_gemm_a8" if layers[0].fused_a8 else "sq_encode + sq_gemm") + " for each of the four linears",
                   "gemm_mode": ("the encode kernel also writes the merged 8-bit activations (M*K bytes), gemm_kernel consumes them: two launches per linear" if layers[0].fused_a8 else "sq_gemm with a workspace: expand_a8_kernel writes the merged 8-bit activations once (M*K bytes), gemm_kernel consumes them") + "; the gemm_fused block times plain sq_gemm, whose sparse part runs inside the GEMM kernel",
                   "l2": "inputs larger than L2 (packed weights + activations + outputs of a step ~2.5 GB)",
                   "sharding": "tokens (M) per rank, weights replicated, no data-path collective"},
        "clocks": clk,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps,
                "note": "pinned host buffers; copies in, kernels and copies out on three streams (PCIe-bound)"},
        # sq_encode + sq_gemm per linear, plus the second kernel a workspace brings with it (activation
        # expansion above 128 rows, split-K finish at or below)
        "gpu_launches": sum(l.launches for l in layers) * args.steps,
        "roofline": {"kernel": "sq_gemm", "bound": "tensor", "achieved": gemm_tops, "peak": int8_peak,
                     "unit": "TOPS", "frac": gemm_tops / int8_peak,
                     "peak_source": f"2 x {peaks['source']} bf16 burst ({peaks['bf16_tflops']} TFLOP/s); INT8:bf16 nominal ratio 2",
                     "frac_of_sustained": gemm_tops / (peaks["bf16_tflops_sustained"] * INT8_OVER_BF16),
                     "frac_of_nominal_4500": gemm_tops / 4500.0,
                     "avg_launch_ms": gemm_ms / n_gemm, "launches": n_gemm,
                     "algorithmic_bytes_per_launch": sum(l.gemm_bytes for l in layers) / len(layers),
                     # the timed mode reads the 8-bit copy of the activations (and, without the fused encode, writes it too)
                     "bytes_per_launch_incl_8bit_copy": sum(l.gemm_bytes + (1.0 if l.fused_a8 else 2.0) * l.M * l.K for l in layers) / len(layers),
                     "traffic": sum(l.gemm_bytes for l in layers) / len(layers)
                     * GEMM_CAPTURE_TRAFFIC_BYTES / GEMM_CAPTURE_ALGO_BYTES,
                     "traffic_note": "EXTRAPOLATED: ncu DRAM bytes of a captured M=2048 launch (whose 8-bit copy stayed in L2) scaled by algorithmic bytes; the kernel is tensor-bound, traffic < algorithmic bytes (see profiles/)"},
        "roofline_encode_in_step": {"kernel": "sq_encode", "bound": "hbm", "achieved": enc_gbs,
                                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": enc_gbs / peaks["hbm_gbs"],
                                    "peak_source": peaks["source"], "traffic": None},
    }
    if rank == 0:
        if not args.no_encode_bench:
            del host_X, host_out
            if not args.no_sweep:
                line["format_sweep"] = {"workload": "M=4096, K=N=8192; b x k/b x {dynamic, static, static with independent scales, fp8/fp4 dynamic, fp8/fp4 static} x outlier channels x{10,50}; Student-t nu=3, 1% outlier channels; rel_err = ||out - fp32(X W^T)||_F / ||fp32(X W^T)||_F; fp8/fp4 rows: TFLOPS on the FP8 tensor path, same denominator",
                                        **bench_format_sweep(sq, dev, peaks)}
            line["gemm_8b_dynamic"] = {"workload": "8B-decoder-shaped linears + the single-GEMM configuration (last row), b=64, k=8, dynamic; median of 20 CUDA-event pairs (small inputs may sit in L2); fused = plain sq_gemm without a workspace",
                                       **bench_8b_dynamic(sq, dev, peaks)}
            line["encode"] = {"workload": "sq_encode alone: bf16 8192 x 8192, Student-t nu=3, 0.5% channels x50, b=64; 3 inputs in rotation (> L2); median of 50 launches",
                              "observed_bound": "dynamic: integer/logic pipe (ncu: 67% busy at 9.4 of 17.5 lane-instructions per element, DRAM 35%); static: at the memory's rate between a launch's first and last round of rows (a row group never waits for data after its first row), no pipe above 58%",
                              **bench_encode_only(sq, dev, peaks)}
            line["gemm_fused"] = {"workload": "70B-shaped linears, M=4096, b=128, k=16: plain sq_gemm (sparse part inside the GEMM kernel) vs the workspace call",
                                  **bench_gemm_fused(sq, layers, dev, peaks)}
            line["decode_static"] = {"workload": "8B-decoder-shaped linears, 1 and 16 tokens, b=64, k=8, STATIC positions (the weight-streaming kernel with one shared row of places)",
                                     **bench_decode_static(sq, dev, peaks)}
            line["weights_sq"] = {"workload": "weights in SQ-format (implicit mask, b=64, k=8) x per-token INT8 activations, 8B-decoder shapes, 1 and 4 tokens",
                                  **bench_weights_sq(sq, dev, peaks)}
            line["producer_fusion"] = {"workload": "sq_rmsnorm_encode: bf16 [M,K] Student-t nu=3, 0.5% channels x50, static positions; GBps = (2 + 0.5 + k/b) bytes per element over the fused call (the unfused pair moves 4 more: the normalised tensor written and read back); median of 30 launches",
                                       **bench_producer_fusion(sq, dev, peaks)}
            lp = bench_layer_prefill(sq, layers, dev)
            if lp is not None:
                line["layer_prefill"] = {"workload": "the step's four 70B-shaped linears (M=4096, b=128, k=16 static) with the two layer normalisations of a decoder layer (inputs of the QKV and gate-up projections)", **lp}
            same = bench_same_run_int8(dev)
            burst, sustained, fp8_burst = bench_int8_tensor_rate(sq)
            line["same_run"] = {"int8_gemm_TOPS": None if same is None else round(same, 1),
                                "what": "torch._int_mm M=4096 N=K=8192 (vendor INT8 GEMM, yardstick only)",
                                "roofline_frac_of_same_run_int8": None if same is None else round(gemm_tops / same, 3),
                                "int8_mma_only_TOPS": round(burst, 1), "int8_mma_only_sustained_TOPS": round(sustained, 1),
                                "mma_only_what": "sq_probe_int8_tensor_rate (and sq_probe_fp8_tensor_rate for kind::f8f6f4): tcgen05.mma 128x256x32 on resident operands, nothing else, one CTA per SM; ~5 ms launches (median of 5) and one ~0.25 s launch; fp_gemm_frac = [slowest, fastest] fp8/fp4 row of format_sweep over the fp8 rate",
                                "fp8_mma_only_TFLOPS": round(fp8_burst, 1),
                                "roofline_frac_of_mma_only": round(gemm_tops / burst, 3),
                                "roofline_frac_of_mma_only_sustained": round(gemm_tops / sustained, 3)}
            line["roofline"]["frac_of_mma_only_same_run"] = round(gemm_tops / burst, 3)
            if "format_sweep" in line:
                fp_tops = [r[5] for r in line["format_sweep"]["rows"] if str(r[2]).startswith("fp8")]
                line["same_run"]["fp_gemm_frac_of_fp8_mma_only"] = [round(min(fp_tops) / fp8_burst, 3), round(max(fp_tops) / fp8_burst, 3)]
        if not args.no_cpu_baseline and world == 1:
            K, N = SHAPES_70B[1]
            ops = dt = 0.0
            cores = 1
            t_end = time.time() + 12.0
            n = 0
            while time.time() < t_end or n == 0:
                o, d, cores = oracle_sample(K, N, BANK_70B, K_70B, 0, rows=128, cols=1024)
                ops, dt, n = ops + o, dt + d, n + 1
            line["cpu_baseline"] = {"value": ops / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n} x (encode + GEMM of 128 token rows x 1024 output channels of the (K,N)=({K},{N}) linear)"}
        # one line; the blocks a reader needs first go LAST (a captured tail then still holds them)
        tail_keys = ["gemm_fused", "encode", "same_run", "roofline_encode_in_step", "gpu_launches", "clocks", "e2e",
                     "cpu_baseline", "roofline"]
        line = {**{k: v for k, v in line.items() if k not in tail_keys}, **{k: line[k] for k in tail_keys if k in line}}
        print(json.dumps(line, separators=(",", ":")))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--m", type=int, default=M_70B, help="tokens per GPU (default: the workload's 4096)")
    ap.add_argument("--linears", type=str, default="",
                    help="comma-separated indices into the four linears (default: all four; a subset is for profiling)")
    ap.add_argument("--no-encode-bench", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the format-parameter sweep block")
    ap.add_argument("--separate-expand", action="store_true",
                    help="step = sq_encode + sq_gemm with a workspace (a separate kernel expands the merged 8-bit operand) instead of sq_encode_a8 + sq_gemm_a8")
    ap.add_argument("--independent-scales", action="store_true",
                    help="run the step with the independent-scale variant of the static format (not the headline)")
    ap.add_argument("--profile-case", choices=PROFILE_CASES, default=None,
                    help="run a few launches of one kernel on a small case and exit (the command profiler captures are taken of)")
    args = ap.parse_args()
    if args.profile_case:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
