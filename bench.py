#!/usr/bin/env python
"""Benchmark of the WHT + diagonal-affine path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload training|prefill|large|tiny]
                    [--impl ours|reference] [--no-sections]

A step is one pass of the whole path over one batch: the forward call
(y = a (.) (x H)/sqrt(d) + b) followed by the backward call (dx, da, db).  The
default workload is the training shape (65536 rows, d = 2048, bf16 rows, fp32
parameters), whose 1 GiB working set is far larger than L2, so no flush is needed
between iterations.  Rank 0 prints ONE JSON line.  With N > 1 ranks every rank
transforms its own rows (rows are independent; weak scaling) and the only exchange
is one all-reduce of da|db per step.

`--impl reference` times the fp64 CPU oracle (the parity authority, a deliberately
slow dense product) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2603_08343_b200 import dp
from paper_2603_08343_b200 import workloads as wl

METRIC = "wht_affine_tokens_per_s_fwd_bwd"
UNIT = "tokens/s"
# DRAM bytes of one launch of the dominant kernel come from the ncu capture recorded in this file, in a
# line "traffic_record: ..." that also names the kernel and a digest of the sources it was built from.
TRAFFIC_PROFILE = os.path.join("profiles", "umma64_bwd_training_d2048.txt")


def ncu_traffic(workload: str, rows: int):
    """(bytes or None, where it comes from): dram__bytes_read.sum + dram__bytes_write.sum of one launch of the
    dominant kernel, read from the committed ncu summary; None once the kernel's sources have changed since."""
    from paper_2603_08343_b200 import build as _build
    path = os.path.join(ROOT, TRAFFIC_PROFILE)
    try:
        text = open(path).read()
    except OSError:
        return None, f"{TRAFFIC_PROFILE} missing"
    for line in text.splitlines():
        if not line.startswith("traffic_record:"):
            continue
        rec = dict(kv.split("=", 1) for kv in line.split()[1:])
        if rec.get("workload") != workload or int(rec.get("rows", -1)) != rows:
            continue
        if rec.get("sources_sha256") != _build.source_digest(rec.get("sources", "").split(",")):
            return None, f"{TRAFFIC_PROFILE}: stale (the sources of {rec.get('kernel')} changed since the capture)"
        total = int(rec["dram_bytes_read"]) + int(rec["dram_bytes_write"])
        return total, f"{TRAFFIC_PROFILE}: {rec.get('kernel')}, one ncu pass at {rows} rows, sources unchanged since"
    return None, f"{TRAFFIC_PROFILE}: no capture recorded for {workload} at {rows} rows"


# ----------------------------------------------------------------------------- helpers

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu_index), "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop_all(self):
        """Ends the sampling; returns every (time, line) sample for summarise()."""
        if self.proc is None:
            return []
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        return list(self.lines)

    @staticmethod
    def summarise(samples, t0=None, t1=None):
        """Median SM clock, maximum power and the throttle reasons seen between t0 and t1."""
        if not samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        sm, mx, reasons, power = [], [], set(), []
        for ts, line in samples:
            if t0 is not None and not (t0 + 0.02 <= ts <= t1 + 0.02):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {
            "sm_mhz": statistics.median(sm) if sm else None,
            "sm_max_mhz": max(mx) if mx else None,
            "power_w_max": max(power) if power else None,
            "samples": len(sm),
            "reasons": sorted(reasons),
        }


def f64(t: torch.Tensor) -> np.ndarray:
    import oracle
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return oracle.widen_bf16_bits(t.view(torch.int16).numpy().view(np.uint16))
    return t.numpy().astype(np.float64)


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def oracle_step_seconds(w: wl.Workload, rows: int, repeats: int = 1):
    """Times the oracle's forward (+ backward when the workload has one) on `rows` rows."""
    import oracle
    ws = w.with_rows(rows)
    x = f64(wl.gen_full(ws, "x"))
    a, b = (f64(t) for t in wl.gen_params(ws))
    dy = f64(wl.gen_full(ws, "dy")) if w.has_bwd else None
    oracle.sylvester_hadamard(w.d)  # the constant matrix is built outside the timed region
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        oracle.wht_affine_fwd(x, a, b)
        if dy is not None:
            oracle.wht_affine_bwd(dy, x, a)
        best = min(best, time.perf_counter() - t0)
    return best


# ----------------------------------------------------------------------------- reference arm

def run_reference(args, rank: int, world: int):
    if rank != 0:
        return
    w = wl.CONFIGS[args.workload]
    # keep the whole run to about a minute of CPU work whatever K is: a short pilot gives the rate, the
    # rows per step follow from it (the per-row cost is constant)
    pilot = {"tiny": 64, "prefill": 2048, "training": 1024, "large": 128}[args.workload]
    rate = pilot / oracle_step_seconds(w, pilot, repeats=2)
    rows = max(16, min(w.T, 16384, int(rate * 60.0 / max(args.steps, 1)) // 16 * 16))
    for _ in range(min(args.warmup, 3)):
        oracle_step_seconds(w, min(rows, 64))
    times = [oracle_step_seconds(w, rows) for _ in range(args.steps)]
    total = sum(times)
    value = rows * args.steps / total
    cores = blas_threads()
    sample = f"{rows} rows of the {w.name} workload per step (d={w.d}), fp64 dense product, fwd{'+bwd' if w.has_bwd else ''}"
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "T_sample": rows, "d": w.d},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


# ----------------------------------------------------------------------------- our arm

class Timer:
    def __init__(self):
        self.start = torch.cuda.Event(enable_timing=True)
        self.end = torch.cuda.Event(enable_timing=True)

    def __enter__(self):
        self.start.record()
        return self

    def __exit__(self, *exc):
        self.end.record()

    def ms(self):
        self.end.synchronize()
        return self.start.elapsed_time(self.end)


def time_loop(fn, iters: int, warmup: int = 3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    with Timer() as t:
        for _ in range(iters):
            fn()
    return t.ms() / iters


def graph_of(fn, repeats: int):
    """CUDA graph of `repeats` back-to-back calls of fn on a side stream (the device time per call without
    the Python launch path, which at ~10 us per call would otherwise bound a 12 us kernel)."""
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(repeats):
                fn()
    return g, s


def section_prefill(B, hbm_peak):
    """Prefill forward; 16 buffer pairs (1 GiB) are rotated so every call misses L2.  Timed as a CUDA graph
    of 64 calls (4 rounds over the buffers) replayed for about a second, and from a plain stream loop."""
    w = wl.CONFIGS["prefill"]
    a, b = (t.cuda() for t in wl.gen_params(w))
    x0 = wl.gen_full(w, "x").cuda()
    nbuf = 16
    xs = [x0.clone() for _ in range(nbuf)]
    ys = [torch.empty_like(x0) for _ in range(nbuf)]
    state = {"i": 0}

    def call():
        i = state["i"] % nbuf
        state["i"] += 1
        B.wht_affine_fwd(xs[i], a, b, ys[i], w.T, w.d, w.dtype)

    def copy():
        i = state["i"] % nbuf
        state["i"] += 1
        B.wht_copy_rows(xs[i], ys[i], w.T, w.d, w.dtype)

    def torch_copy():
        i = state["i"] % nbuf
        state["i"] += 1
        ys[i].copy_(xs[i])

    per_graph = 4 * nbuf
    out = {"T": w.T, "d": w.d, "dtype": "bf16", "l2": "16 rotating buffer pairs (1 GiB)",
           "timing": f"CUDA graph of {per_graph} calls replayed; stream_loop: plain Python launches"}
    gb = 2 * w.T * w.d * w.io_bytes / 1e9
    for key, fn in (("fwd", call), ("copy_rows", copy), ("torch_copy", torch_copy)):
        g, s = graph_of(fn, per_graph)
        with torch.cuda.stream(s):
            burst = time_loop(g.replay, 1, warmup=1) / per_graph
            reps = max(3, int(math.ceil((0.6 if key == "fwd" else 0.15) * 1e3 / (burst * per_graph))))
            ms = time_loop(g.replay, reps, warmup=1) / per_graph
        out[f"{key}_us"] = 1e3 * ms
        out[f"{key}_GBps"] = gb / (ms * 1e-3)
        if key == "fwd":
            out["fwd_burst_us"] = 1e3 * burst
    ms = out["fwd_us"] * 1e-3
    out.update({"fwd_tokens_per_s": w.T / (ms * 1e-3), "fwd_frac_of_measured_peak": gb / (ms * 1e-3) / hbm_peak,
                "fwd_frac_of_8000": gb / (ms * 1e-3) / 8000.0})
    out["fwd_stream_loop_us"] = 1e3 * time_loop(call, 20 * nbuf, warmup=nbuf)
    out["fwd_us_l2_warm"] = 1e3 * time_loop(lambda: B.wht_affine_fwd(xs[0], a, b, ys[0], w.T, w.d, w.dtype), 200, warmup=10)
    return out


def section_decode(B):
    w0 = wl.CONFIGS["decode"]
    a, b = (t.cuda() for t in wl.gen_params(w0))
    out = {}
    for T in wl.DECODE_T:
        w = w0.with_rows(T)
        x = wl.gen_full(w, "x").cuda()
        y = torch.empty_like(x)
        fn = lambda: B.wht_affine_fwd_decode(x, a, b, y, w.T, w.d, w.dtype)  # noqa: E731
        loop_us = 1e3 * time_loop(fn, 2000, warmup=20)
        # the same call with its arguments marshalled once (binding.prepare): what a decode loop would use
        prepared_us = 1e3 * time_loop(B.prepare("wht_affine_fwd_decode", x, a, b, y, w.T, w.d, w.dtype), 4000, warmup=20)
        # CUDA-graph replay of 50 back-to-back calls: per-call device time without launch overhead
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for _ in range(3):
                B.wht_affine_fwd_decode(x, a, b, y, w.T, w.d, w.dtype)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(50):
                    B.wht_affine_fwd_decode(x, a, b, y, w.T, w.d, w.dtype)
            graph_us = 1e3 * time_loop(g.replay, 40, warmup=3) / 50
        out[f"T{T}"] = {"stream_loop_us_per_call": loop_us, "prepared_stream_loop_us_per_call": prepared_us,
                        "graph_replay_us_per_call": graph_us}
    out["d"] = w0.d
    return out


def section_tiny(B):
    """The Tiny config (64 x 256, fp32): latency-bound; device time per call from a CUDA-graph replay of 50
    forward + backward pairs (the backward is its main kernel plus the small second pass)."""
    w = wl.CONFIGS["tiny"]
    x, dy = wl.gen_full(w, "x").cuda(), wl.gen_full(w, "dy").cuda()
    a, b = (t.cuda() for t in wl.gen_params(w))
    y, dx = torch.empty_like(x), torch.empty_like(x)
    da, db = torch.empty(w.d, device="cuda"), torch.empty(w.d, device="cuda")
    ws = torch.empty(max(B.wht_affine_bwd_workspace_bytes(w.T, w.d, w.dtype), 16), dtype=torch.uint8, device="cuda")
    out = {"T": w.T, "d": w.d, "dtype": "fp32"}
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for which in ("fwd", "bwd"):
            def call():
                if which == "fwd":
                    B.wht_affine_fwd(x, a, b, y, w.T, w.d, w.dtype)
                else:
                    B.wht_affine_bwd_ws(dy, x, a, dx, da, db, w.T, w.d, w.dtype, ws)
            for _ in range(3):
                call()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(50):
                    call()
            out[f"{which}_graph_replay_us_per_call"] = 1e3 * time_loop(g.replay, 40, warmup=3) / 50
    return out


def section_paper_shapes(B, hbm_peak):
    """The paper's own inference shapes (its prefill table: batch 1024 x 64 tokens = 65536 rows; its
    decode table: batch 2048, one row per sequence and step) at its two power-of-two model widths."""
    out = {}
    for d in (1024, 2048):
        w = wl.Workload("paper", 1024 * 64, d, wl.WHT_BF16, "normal", 10 + d, False, "")
        a, b = (t.cuda() for t in wl.gen_params(w))
        x = wl.gen_full(w.with_rows(8192), "x").cuda().repeat(8, 1)
        y = torch.empty_like(x)
        ms = time_loop(lambda: B.wht_affine_fwd(x, a, b, y, w.T, w.d, w.dtype), 50, warmup=5)
        gb = 2 * w.T * w.d * 2 / 1e9
        entry = {"prefill_T": w.T, "prefill_fwd_us": 1e3 * ms, "prefill_fwd_GBps": gb / (ms * 1e-3),
                 "prefill_frac_of_measured_peak": gb / (ms * 1e-3) / hbm_peak,
                 "prefill_tokens_per_s": w.T / (ms * 1e-3)}
        xd = x[:2048].contiguous()
        yd = torch.empty_like(xd)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for _ in range(3):
                B.wht_affine_fwd_decode(xd, a, b, yd, 2048, d, w.dtype)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                for _ in range(50):
                    B.wht_affine_fwd_decode(xd, a, b, yd, 2048, d, w.dtype)
            entry["decode_T"] = 2048
            entry["decode_graph_replay_us_per_call"] = 1e3 * time_loop(g.replay, 40, warmup=3) / 50
        out[f"d{d}"] = entry
        del x, y
    return out


def section_tensor_parallel_local(B, hbm_peak):
    """Column-sharded calls of ONE rank with every rank's block in this GPU's memory (the kernels read the
    blocks through a pointer table; on several GPUs the other entries are peer mappings and the NVLink
    transfer, not the kernel, sets the time).  Bytes: (g+1) blocks forward, (2g+1) backward."""
    from paper_2603_08343_b200 import tp
    out = {}
    for g, w_, T in ((2, 1024, 65536), (4, 1024, 32768), (8, 1024, 16384), (8, 256, 65536)):
        wk = wl.Workload("tp", T, w_, wl.WHT_BF16_PF32, "normal", 20 + g, True, "")
        base = wl.gen_full(wk.with_rows(4096), "x").cuda()
        xs = [base.roll(s, 0).repeat(T // 4096, 1) for s in range(g)]
        dys = [base.roll(s + g, 0).repeat(T // 4096, 1) for s in range(g)]
        a, b = (t.cuda() for t in wl.gen_params(wk))
        as_ = [a.clone() for _ in range(g)]
        rank = tp.TpWht(g, g - 1)
        y = torch.empty_like(xs[0])
        f_ms = time_loop(lambda: rank.forward(xs, a, b, T, w_, out=y), 20, warmup=5)
        b_ms = time_loop(lambda: rank.backward(dys, xs, as_, T, w_), 20, warmup=5)
        fb, bb = (g + 1) * T * w_ * 2 / 1e9, (2 * g + 1) * T * w_ * 2 / 1e9
        out[f"g{g}_w{w_}"] = {"T": T, "fwd_us": 1e3 * f_ms, "fwd_GBps": fb / (f_ms * 1e-3),
                             "fwd_frac_of_measured_peak": fb / (f_ms * 1e-3) / hbm_peak,
                             "bwd_us": 1e3 * b_ms, "bwd_GBps": bb / (b_ms * 1e-3),
                             "bwd_frac_of_measured_peak": bb / (b_ms * 1e-3) / hbm_peak}
        del xs, dys, y, base
    return out


def section_other_shapes(B, hbm_peak):
    """Shapes outside the five configs, 256 MiB per row tensor: fp32 storage (butterfly kernels at d <= 512 in
    the forward, streamed mma.sync kernels otherwise) and the block-diagonal form."""
    out = {}
    for d in (256, 512, 1024, 2048, 4096):
        T = (256 << 20) // (4 * d)
        x = torch.randn(T, d, device="cuda")
        a = torch.rand(d, device="cuda") + 0.5
        y = torch.empty_like(x)
        da, db = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
        f_ms = time_loop(lambda: B.wht_affine_fwd(x, a, a, y, T, d, wl.WHT_F32), 20, warmup=5)
        b_ms = time_loop(lambda: B.wht_affine_bwd(x, x, a, y, da, db, T, d, wl.WHT_F32), 20, warmup=5)
        out[f"fp32_d{d}"] = {"T": T, "fwd_us": 1e3 * f_ms, "fwd_frac_of_measured_peak": 8 * T * d / (f_ms * 1e6) / hbm_peak,
                            "bwd_us": 1e3 * b_ms, "bwd_frac_of_measured_peak": 12 * T * d / (b_ms * 1e6) / hbm_peak}
        del x, y
    for d, block in ((768, 256), (1536, 512)):
        T = 65536
        x = torch.randn(T, d, device="cuda").bfloat16()
        a = torch.rand(d, device="cuda") + 0.5
        y = torch.empty_like(x)
        da, db = torch.empty(d, device="cuda"), torch.empty(d, device="cuda")
        ws = torch.empty(max(B.wht_affine_bwd_grouped_workspace_bytes(T, d, block, wl.WHT_BF16_PF32), 16),
                         dtype=torch.uint8, device="cuda")
        f_ms = time_loop(lambda: B.wht_affine_fwd_grouped(x, a, a, y, T, d, block, wl.WHT_BF16_PF32), 20, warmup=5)
        b_ms = time_loop(lambda: B.wht_affine_bwd_grouped(x, x, a, y, da, db, T, d, block, wl.WHT_BF16_PF32, ws),
                         20, warmup=5)
        out[f"grouped_d{d}"] = {"T": T, "block": block, "fwd_us": 1e3 * f_ms,
                               "fwd_frac_of_measured_peak": 4 * T * d / (f_ms * 1e6) / hbm_peak,
                               "bwd_us": 1e3 * b_ms, "bwd_frac_of_measured_peak": 6 * T * d / (b_ms * 1e6) / hbm_peak}
        del x, y
    return out


def burst_and_sustained(fn, min_seconds: float, gpu_index: int = 0):
    """(burst ms, sustained ms, median SM MHz of the sustained loop): 30 launches after a one-second pause,
    then a loop of at least `min_seconds` of device time."""
    for _ in range(5):
        fn()
    torch.cuda.synchronize()
    time.sleep(1.0)
    burst = time_loop(fn, 30, warmup=0)
    n = max(30, int(math.ceil(min_seconds * 1e3 / burst)))
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.1)
    t0 = time.time()
    ms = time_loop(fn, n, warmup=0)
    torch.cuda.synchronize()
    t1 = time.time()
    clk = ClockSampler.summarise(sampler.stop_all(), t0 + 0.2 * (t1 - t0), t1)
    return burst, ms, clk["sm_mhz"]


def section_fwd_bwd(B, name, hbm_peak, min_seconds):
    """Forward and backward timed separately on a workload larger than L2: in a burst and sustained."""
    w = wl.CONFIGS[name]
    base_rows = min(w.T, 8192)
    a, b = (t.cuda() for t in wl.gen_params(w))
    xb = wl.gen_full(w.with_rows(base_rows), "x").cuda()
    dyb = wl.gen_full(w.with_rows(base_rows), "dy").cuda()
    reps = w.T // base_rows
    x = xb.repeat(reps, 1)
    dy = dyb.repeat(reps, 1)
    del xb, dyb
    y = torch.empty_like(x)
    da = torch.empty(w.d, dtype=torch.float32, device="cuda")
    db = torch.empty_like(da)
    fb = 2 * w.T * w.d * w.io_bytes / 1e9
    bb = 3 * w.T * w.d * w.io_bytes / 1e9
    res = {"T": w.T, "d": w.d, "rows_drawn": base_rows, "rows_tiled": reps,
           "timing": f"burst: 30 launches after a pause; plain: a loop of >= {min_seconds:g} s"}
    for which, fn, gb in (("fwd", lambda: B.wht_affine_fwd(x, a, b, y, w.T, w.d, w.dtype), fb),
                          ("bwd", lambda: B.wht_affine_bwd(dy, x, a, y, da, db, w.T, w.d, w.dtype), bb)):
        burst, ms, mhz = burst_and_sustained(fn, min_seconds)
        res.update({f"{which}_us": 1e3 * ms, f"{which}_GBps": gb / (ms * 1e-3),
                    f"{which}_frac_of_measured_peak": gb / (ms * 1e-3) / hbm_peak,
                    f"{which}_frac_of_8000": gb / (ms * 1e-3) / 8000.0, f"{which}_tokens_per_s": w.T / (ms * 1e-3),
                    f"{which}_sm_mhz": mhz, f"{which}_burst_us": 1e3 * burst,
                    f"{which}_burst_frac_of_measured_peak": gb / (burst * 1e-3) / hbm_peak})
    if w.dtype != wl.WHT_F32:
        # the backward with g carried into the second product as a bf16 pair (dx rounded once)
        B.wht_affine_set_bwd_operand_mode(1)
        try:
            burst, ms, mhz = burst_and_sustained(lambda: B.wht_affine_bwd(dy, x, a, y, da, db, w.T, w.d, w.dtype),
                                                 min_seconds)
        finally:
            B.wht_affine_set_bwd_operand_mode(0)
        res.update({"bwd_pair_mode_us": 1e3 * ms, "bwd_pair_mode_frac_of_measured_peak": bb / (ms * 1e-3) / hbm_peak,
                    "bwd_pair_mode_sm_mhz": mhz, "bwd_pair_mode_burst_us": 1e3 * burst})
    iters = 50
    c_ms = time_loop(lambda: B.wht_copy_rows(x, y, w.T, w.d, w.dtype), iters, warmup=10)
    r_ms = time_loop(lambda: B.wht_affine_fwd_residual(x, a, b, dy, y, w.T, w.d, w.dtype), iters, warmup=10)
    res.update({"copy_rows_GBps": fb / (c_ms * 1e-3),
                # forward fused with the residual add: reads x and the residual stream, writes y (3 row tensors)
                "fwd_residual_us": 1e3 * r_ms, "fwd_residual_GBps": bb / (r_ms * 1e-3),
                "fwd_residual_frac_of_measured_peak": bb / (r_ms * 1e-3) / hbm_peak})
    # the dense projection this path replaces, as context: cuBLAS bf16 [T x d] x [d x d]
    if w.dtype != wl.WHT_F32:
        wmat = torch.randn(w.d, w.d, device="cuda", dtype=torch.bfloat16)
        g_ms = time_loop(lambda: torch.matmul(x, wmat, out=y), 12)
        res["dense_gemm_bf16_us"] = 1e3 * g_ms
        res["dense_gemm_tflops"] = 2.0 * w.T * w.d * w.d / (g_ms * 1e-3) / 1e12
    return res


def run_ours(args, rank: int, world: int, local_rank: int):
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2603_08343_b200 import build as _build
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    from paper_2603_08343_b200 import binding as B
    if args.variant:
        B.wht_affine_set_variant(args.variant)

    hbm_peak, peak_src = load_peaks()
    w = wl.CONFIGS[args.workload]
    if args.rows:
        w = w.with_rows(args.rows)  # a smaller case of the same kernels (profiler captures)
    if args.fp32_rows:  # the same shape stored as fp32 (profiler captures of the fp32 kernels)
        w = wl.Workload(w.name, w.T, w.d, wl.WHT_F32, w.dist, w.seed, w.has_bwd, w.note)
    # every rank draws its own rows (weak scaling): the seed is offset by the rank
    wr = wl.Workload(w.name, w.T, w.d, w.dtype, w.dist, w.seed + 1000 * rank, w.has_bwd, w.note)
    base_rows = min(w.T, 8192) if w.dist != "normal" else w.T
    a_h, b_h = wl.gen_params(wr)
    x_h = wl.gen_full(wr.with_rows(base_rows), "x", threads=16)
    dy_h = wl.gen_full(wr.with_rows(base_rows), "dy", threads=16) if w.has_bwd else None
    reps = w.T // base_rows
    a, b = a_h.cuda(), b_h.cuda()
    x = x_h.cuda().repeat(reps, 1)
    dy = dy_h.cuda().repeat(reps, 1) if w.has_bwd else None
    y = torch.empty_like(x)
    dx = torch.empty_like(x) if w.has_bwd else None
    # da|db, contiguous: one all-reduce per step, left in flight while the next step's forward runs (two buckets
    # in turn; the sum is waited for when its bucket comes round again and before a timed region ends)
    ring = dp.GradBucketRing(w.d, device="cuda", n=2)
    da, db = ring.buckets[0].da, ring.buckets[0].db  # for the per-call loops below

    # small working sets are rotated through enough buffers to exceed L2 (126 MB)
    step_bytes = (4 if w.has_bwd else 2) * w.T * w.d * w.io_bytes
    nbuf = 1 if step_bytes > 400e6 else int(np.ceil(1.0e9 / step_bytes))
    xs, ys, dys, dxs = [x], [y], [dy], [dx]
    for _ in range(nbuf - 1):
        xs.append(x.clone())
        ys.append(torch.empty_like(x))
        dys.append(dy.clone() if w.has_bwd else None)
        dxs.append(torch.empty_like(x) if w.has_bwd else None)
    l2_note = ("working set %.0f MB per step, larger than L2" % (step_bytes / 1e6)) if nbuf == 1 else \
        f"{nbuf} rotating buffer sets ({nbuf * step_bytes / 1e6:.0f} MB), larger than L2"
    counter = {"i": 0}
    launches_per_step = 1 + (2 if w.has_bwd else 0)

    def step(ev=None):
        i = counter["i"] % nbuf
        counter["i"] += 1
        if ev is not None:
            ev[0].record()
        B.wht_affine_fwd(xs[i], a, b, ys[i], w.T, w.d, w.dtype)
        if ev is not None:
            ev[1].record()
        if w.has_bwd:
            bucket = ring.acquire()
            B.wht_affine_bwd(dys[i], xs[i], a, dxs[i], bucket.da, bucket.db, w.T, w.d, w.dtype)
            if ev is not None:
                ev[2].record()
            ring.all_reduce_async(bucket)  # the path's only exchange; nothing to do on one rank

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    def max_over_ranks(ms: float) -> float:
        if world == 1:
            return ms
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def timed(fn, n: int):
        """n calls back to back between two CUDA events (nothing in between, so that each kernel may start
        while its predecessor drains), barrier + synchronize on both sides, max over ranks; also the
        wall-clock window for the clock samples."""
        sync_all()
        t0 = time.time()
        with Timer() as t:
            for _ in range(n):
                fn()
            ring.drain()  # the last steps' all-reduces belong to the timed region
        ms = t.ms()
        torch.cuda.synchronize()
        t1 = time.time()
        if world > 1:
            dist.barrier()
        return max_over_ranks(ms), (t0, t1)

    def count_for(seconds: float, ms_per_call: float, at_least: int) -> int:
        return max(at_least, int(math.ceil(seconds * 1e3 / max(ms_per_call, 1e-6))))

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    # 1. burst: K steps straight after the warm-up, the GPU still at its idle clocks and temperature
    burst_ms, burst_win = timed(step, args.steps)
    # 2. sustained: the same step repeated for at least --min-seconds of device time (the state a training
    #    loop is in: the board's power limit has settled the SM clock) ...
    n_long = count_for(args.min_seconds, burst_ms / args.steps, args.steps)
    long_ms, long_win = timed(step, n_long)
    # 3. ... and, with no pause, exactly K steps more: the headline figure (ms_per_step, value)
    total_ms, head_win = timed(step, args.steps)
    ms_per_step = total_ms / args.steps
    value = world * w.T / (ms_per_step * 1e-3)

    # per-call durations for the roofline figure: launches of one call back to back between two events
    def fwd_only():
        i = counter["i"] % nbuf
        counter["i"] += 1
        B.wht_affine_fwd(xs[i], a, b, ys[i], w.T, w.d, w.dtype)

    def bwd_only():
        i = counter["i"] % nbuf
        counter["i"] += 1
        B.wht_affine_bwd(dys[i], xs[i], a, dxs[i], da, db, w.T, w.d, w.dtype)

    def call_figures(fn, bytes_per_launch):
        """Burst (after a one-second pause, 30 launches) and sustained (>= --min-seconds) time of one call."""
        for _ in range(3):
            fn()
        sync_all()
        time.sleep(1.0)
        n_burst = 30
        b_ms, b_win = timed(fn, n_burst)
        n = count_for(args.min_seconds, b_ms / n_burst, n_burst)
        l_ms, l_win = timed(fn, n)
        return {"burst_ms": b_ms / n_burst, "burst_launches": n_burst, "burst_win": b_win,
                "ms": l_ms / n, "launches": n, "win": l_win, "bytes": bytes_per_launch}

    fwd_fig = call_figures(fwd_only, 2 * w.T * w.d * w.io_bytes)
    bwd_fig = call_figures(bwd_only, 3 * w.T * w.d * w.io_bytes) if w.has_bwd else None
    # the same calls inside the step sequence with an event after every call, for comparison
    # (each event adds a few microseconds of idle front-end time to the call before it)
    ev_steps = min(max(args.steps, 20), 200)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(ev_steps)]
    for k in range(ev_steps):
        step(events[k])
    ring.drain()
    torch.cuda.synchronize()
    fwd_ms = [e[0].elapsed_time(e[1]) for e in events]
    bwd_ms = [e[1].elapsed_time(e[2]) for e in events] if w.has_bwd else []
    samples = sampler.stop_all() if rank == 0 else None

    def clocks_in(win):
        return ClockSampler.summarise(samples, *win) if samples is not None else None

    def call_summary(fig):
        gbps = fig["bytes"] / 1e9 / (fig["ms"] * 1e-3)
        gbps_b = fig["bytes"] / 1e9 / (fig["burst_ms"] * 1e-3)
        ck, ckb = clocks_in(fig["win"]), clocks_in(fig["burst_win"])
        mhz = ck["sm_mhz"] if ck else None
        return {"ms": fig["ms"], "launches": fig["launches"], "GBps": gbps, "frac_of_measured_peak": gbps / hbm_peak,
                "frac_of_nominal_8000": gbps / 8000.0, "tokens_per_s": w.T / (fig["ms"] * 1e-3), "sm_mhz": mhz,
                "us_x_mhz": fig["ms"] * 1e3 * mhz if mhz else None,
                "burst": {"ms": fig["burst_ms"], "launches": fig["burst_launches"], "GBps": gbps_b,
                          "frac_of_measured_peak": gbps_b / hbm_peak, "sm_mhz": ckb["sm_mhz"] if ckb else None}}

    fwd_sum = call_summary(fwd_fig)
    bwd_sum = call_summary(bwd_fig) if w.has_bwd else None
    # the clock record of the headline: the sustained loop and the K timed steps that follow it without a pause
    clocks = clocks_in((long_win[0], head_win[1])) if rank == 0 else None
    if clocks is not None:
        clocks["window"] = f"{n_long} steps of the sustained loop + the {args.steps} timed steps, back to back"
        clocks["burst_steps"] = clocks_in(burst_win)

    # roofline of the dominant call: the backward call when there is one
    dom_sum = bwd_sum if w.has_bwd else fwd_sum
    dom_fig = bwd_fig if w.has_bwd else fwd_fig
    dom = "wht_affine_bwd (main kernel + the small second pass)" if w.has_bwd else "wht_affine_fwd"
    traffic, traffic_source = (ncu_traffic(w.name, w.T) if w.has_bwd and not args.fp32_rows
                               else (None, "no capture recorded for this call"))
    roofline = {"bound": "hbm", "kernel": dom, "achieved": dom_sum["GBps"], "peak": hbm_peak, "unit": "GB/s",
                "frac": dom_sum["frac_of_measured_peak"], "frac_burst": dom_sum["burst"]["frac_of_measured_peak"],
                "peak_source": peak_src, "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic_bytes_per_launch": dom_fig["bytes"], "avg_launch_ms": dom_sum["ms"],
                "launches": dom_sum["launches"], "avg_launch_ms_burst": dom_sum["burst"]["ms"],
                "sm_mhz": dom_sum["sm_mhz"], "sm_mhz_burst": dom_sum["burst"]["sm_mhz"], "us_x_mhz": dom_sum["us_x_mhz"],
                "timing": f"frac: {dom_sum['launches']} launches back to back between two CUDA events (>= "
                          f"{args.min_seconds:g} s: sustained, the board's power limit settles the SM clock); "
                          f"frac_burst: {dom_sum['burst']['launches']} launches after a one-second pause",
                "frac_of_nominal_8000": dom_sum["frac_of_nominal_8000"]}
    fwd_b2b_ms = fwd_sum["ms"]

    # ---- end to end: pinned host buffers in, results back to the host, every step
    e2e = None
    staging = {"x": x, "a": a, "b": b, "y": y, "dy": dy, "dx": dx, "da": da, "db": db}
    e2e_launches = None
    xp, ap, bp = x_h.repeat(reps, 1).pin_memory(), a_h.pin_memory(), b_h.pin_memory()
    yp = torch.empty_like(xp).pin_memory()
    h2d = xp.numel() * xp.element_size() + 2 * ap.numel() * ap.element_size()
    d2h = yp.numel() * yp.element_size()
    if w.has_bwd:
        dyp = dy_h.repeat(reps, 1).pin_memory()
        dxp = torch.empty_like(xp).pin_memory()
        dap = torch.empty(w.d, dtype=torch.float32).pin_memory()
        dbp = torch.empty(w.d, dtype=torch.float32).pin_memory()
        h2d += dyp.numel() * dyp.element_size()
        d2h += dxp.numel() * dxp.element_size() + 8 * w.d

    pipe = B.HostPipe(chunk_rows=max(1024, (32 << 20) // (w.d * w.io_bytes)))

    def e2e_step():
        # x, a, b in -> forward -> y out; dy in -> backward (x still resident) -> dx, da, db out
        B.forward_host(xp, ap, bp, yp, staging, pipe=pipe)
        if w.has_bwd:
            B.backward_host(dyp, xp, ap, dxp, dap, dbp, staging, pipe=pipe, x_resident=True)
        pipe.join()

    e2e_steps = max(2, min(args.steps, 5))
    e2e_ms = time_loop(e2e_step, e2e_steps, warmup=1)
    if world > 1:
        tmax = torch.tensor([e2e_ms], device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        e2e_ms = float(tmax.item())
    e2e = {"value": world * w.T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": e2e_steps,
           "api": "binding.forward_host + binding.backward_host with a HostPipe (pinned host -> device -> C ABI -> "
                  "pinned host; rows move in chunks on two copy streams, x stays resident between the two calls)"}
    del xp, yp, staging
    if w.has_bwd:
        del dyp, dxp
    ring.drain()
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32",  # the arithmetic type; the storage types are in config.storage
        "data": "synthetic",
        "config": {"workload": w.name, "T_per_gpu": w.T, "d": w.d,
                   "storage": {0: "fp32", 1: "bf16 rows, bf16 params", 2: "bf16 rows, fp32 params"}[w.dtype],
                   "step": "wht_affine_fwd + wht_affine_bwd" if w.has_bwd else "wht_affine_fwd",
                   "l2": l2_note, "variant": B.wht_affine_get_variant(),
                   "bwd_operand_mode": B.wht_affine_get_bwd_operand_mode(),
                   "parallelism": f"dp{world} (rows sharded; all-reduce of da|db only, in flight under the next "
                                  f"step's forward)" if world > 1 else "single GPU"},
        "fwd": dict(fwd_sum, ms_in_step_with_events=statistics.mean(fwd_ms)),
        "roofline": roofline, "e2e": e2e, "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        # the same step: straight after the warm-up (burst), and over the long loop the headline follows
        "burst": {"steps": args.steps, "ms_per_step": burst_ms / args.steps,
                  "value": world * w.T / (burst_ms / args.steps * 1e-3)},
        "sustained": {"steps": n_long, "ms_per_step": long_ms / n_long, "seconds": long_ms * 1e-3,
                      "value": world * w.T / (long_ms / n_long * 1e-3)},
        "timed_region": f"{warm} warm-up steps, {args.steps} steps (burst), {n_long} steps (sustained, >= "
                        f"{args.min_seconds:g} s), then without a pause the {args.steps} steps of ms_per_step and value",
    }
    if w.has_bwd:
        out["bwd"] = dict(bwd_sum, ms_in_step_with_events=statistics.mean(bwd_ms))

    # ---- CPU baseline: the oracle as it stands, on a bounded sample of the same workload
    # (a short pilot sizes it: up to 16384 rows per pass, passes until about 12 s of CPU work)
    # On one rank only: with several ranks the line is about scaling, and the other ranks have left.
    if world == 1:
        pilot = {"tiny": 64, "prefill": 4096, "training": 2048, "large": 256}[w.name]
        rate = pilot / oracle_step_seconds(w, pilot)
        rows = min(w.T, 16384, max(pilot, int(rate * 4) // 256 * 256))
        passes = max(1, min(16, math.ceil(12.0 * rate / rows)))
        sec = sum(oracle_step_seconds(w, rows) for _ in range(passes))
        out["cpu_baseline"] = {"value": rows * passes / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                               "seconds": sec,
                               "sample": f"{passes} passes over {rows} rows of the {w.name} workload (d={w.d}), fp64 "
                                         f"dense product, fwd{'+bwd' if w.has_bwd else ''}; tokens/s from that sample "
                                         "(per-row cost is constant)"}

    if not args.no_sections and world == 1:
        del xs, ys, dys, dxs, x, y, dy, dx
        torch.cuda.empty_cache()
        sections = {}
        sections["tiny"] = section_tiny(B)
        sections["prefill"] = section_prefill(B, hbm_peak)
        sections["decode"] = section_decode(B)
        sections["training"] = section_fwd_bwd(B, "training", hbm_peak, args.min_seconds)
        sections["large"] = section_fwd_bwd(B, "large", hbm_peak, args.min_seconds)
        sections["paper_shapes"] = section_paper_shapes(B, hbm_peak)
        sections["tensor_parallel_local"] = section_tensor_parallel_local(B, hbm_peak)
        sections["other_shapes"] = section_other_shapes(B, hbm_peak)
        out["sections"] = sections
        # the figures the target names, one line each: fraction of the measured copy bandwidth and of the
        # nominal 8 TB/s ("burst" = 30 launches after a pause, plain = a loop of >= --min-seconds)
        pc = {}
        pf = sections["prefill"]
        pc["prefill_fwd"] = {"us": pf["fwd_us"], "frac": pf["fwd_frac_of_measured_peak"], "frac_8000": pf["fwd_frac_of_8000"]}
        for name in ("training", "large"):
            sec = sections[name]
            for which in ("fwd", "bwd"):
                pc[f"{name}_{which}"] = {"us": sec[f"{which}_us"], "frac": sec[f"{which}_frac_of_measured_peak"],
                                         "frac_8000": sec[f"{which}_frac_of_8000"], "sm_mhz": sec[f"{which}_sm_mhz"],
                                         "burst_us": sec[f"{which}_burst_us"],
                                         "burst_frac": sec[f"{which}_burst_frac_of_measured_peak"]}
            pc[f"{name}_bwd_pair_mode"] = {"us": sec.get("bwd_pair_mode_us"),
                                           "frac": sec.get("bwd_pair_mode_frac_of_measured_peak")}
            pc[f"{name}_dense_gemm_us"] = sec.get("dense_gemm_bf16_us")
        pc["decode_us_per_call"] = {k: {"graph": v["graph_replay_us_per_call"], "stream_loop": v["stream_loop_us_per_call"],
                                        "prepared_stream_loop": v["prepared_stream_loop_us_per_call"]}
                                    for k, v in sections["decode"].items() if k.startswith("T")}
        out["roofline"]["per_config"] = pc
    print(json.dumps(compact(out)))
    ring.drain()
    if world > 1:
        dist.destroy_process_group()


def compact(obj):
    """Floats to 5 significant digits (the line is long; the driver keeps only its tail)."""
    if isinstance(obj, float):
        return float(f"{obj:.5g}")
    if isinstance(obj, dict):
        return {k: compact(v) for k, v in obj.items()}
    if isinstance(obj, (list, tuple)):
        return [compact(v) for v in obj]
    return obj


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="training", choices=["tiny", "prefill", "training", "large"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--no-sections", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="device time of the sustained loops (the step loop before the timed steps, and the "
                         "per-call loops of the roofline figure)")
    ap.add_argument("--rows", type=int, default=0,
                    help="override the workload's row count (small cases for profiler captures; "
                         "not the benchmark configuration)")
    ap.add_argument("--fp32-rows", action="store_true",
                    help="store the workload's rows and parameters as fp32 (profiler captures; not the "
                         "benchmark configuration)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
