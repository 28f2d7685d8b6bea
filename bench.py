#!/usr/bin/env python
"""Benchmark of the UBP inference path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
                    [--variant V] [--table FILE]

One "step" = one pass of the inference hot path over one batch of synthetic
activations already resident in HBM: a single launch of the layer's kernel
(packing and plan building are the offline model-conversion steps; their
host time is reported separately as pack_ms / plan_ms). The default workload
is the MobileNetV1-shaped pointwise layer 512->512 at 14x14, batch 32, 1x4
blocks, 70 % sparsity, fused bias+ReLU. L2 is flushed between steps (the
26 MB working set would otherwise stay cached).

Prints ONE JSON line (rank 0). With N > 1 (torchrun) every rank runs the
same layer on its own batch (columns are independent: no collective on the
path), value = total work / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import ubp_synth  # noqa: E402

METRIC = "effective GFLOP/s (2 x surviving MACs / time) of one UBP layer"
SM_COUNT, FP32_LANES, SM_MAX_GHZ = 148, 128, 1.965
FP32_PEAK_TFLOPS = SM_COUNT * FP32_LANES * 2 * SM_MAX_GHZ / 1e3     # 74.45: plain FP32 FMA pipes at max clock

WORKLOADS = {
    "mbv1_pw512": dict(cfg="mbv1_pw512", kw={}),
    "fc64": dict(cfg="fc64", kw={}),
    "r50_3x3": dict(cfg="r50_3x3", kw={}),
}
for _nb in (2, 4, 8, 16):
    for _sp in (50, 70, 80, 90, 95):
        WORKLOADS[f"sweep_nb{_nb}_p{_sp}"] = dict(cfg="sweep", kw=dict(Nb=_nb, sparsity_pct=_sp))
for _li in range(13):
    WORKLOADS[f"mbv1_L{_li + 1}"] = dict(cfg="mbv1_chain", kw={}, index=_li)


# Block selection (expansion and division, Section 4.1) on dense weights: M x C x R, block size, sparsity %.
# bed_r50_3x3 is the case Section 5.2 names as the slowest selection of its experiments (ResNet50's largest layers,
# block size 2, 50 % sparsity); bed_mbv1_pw1024 is MobileNetV1's largest pointwise layer at the setting of the
# Section 3.2 example (block size 4, 90 %).
BED_WORKLOADS = {
    "bed_r50_3x3": (512, 512, 9, 2, 50),
    "bed_mbv1_pw1024": (1024, 1024, 1, 4, 90),
    "bed_2048_nb2_p50": (2048, 2048, 1, 2, 50),
    "bed_2048_nb4_p70": (2048, 2048, 1, 4, 70),
}


KMAJOR_B = 4     # kmajor_pw512: the headline layer's shape with blocks of 4 consecutive INPUT channels in one output row


KMAJOR_WORKLOADS = {"kmajor_pw512": 70, "kmajor_pw512_p80": 80, "kmajor_pw512_p90": 90, "kmajor_pw512_p95": 95}


def get_layer(name: str, seed_index: int = 0):
    if name in KMAJOR_WORKLOADS:
        # 512 -> 512 channels at 14 x 14, batch 32, blocks of KMAJOR_B consecutive INPUT channels inside one output row:
        # generated as the transposed layer (blocks run down the rows of [C][M]) and turned round. The Layer object
        # describes it as M*C*(1-p) single weights (Nb = 1); the packed form keeps the runs (build_runner).
        sp = KMAJOR_WORKLOADS[name]
        t = ubp_synth.make_layer(name, 512, 512, KMAJOR_B, sp, 7000 + seed_index, B=32, H=14, Wd=14, w_scale=0.05)
        return ubp_synth.Layer(name, t.C, t.M, 1, 1, sp, t.m * KMAJOR_B, np.ascontiguousarray(t.W.transpose(1, 0, 2)),
                               np.ascontiguousarray(t.mask.T), t.X, t.bias, True, t.B, t.H, t.Wd)
    w = WORKLOADS[name]
    layers = ubp_synth.config_layers(w["cfg"], index=seed_index, **w["kw"])
    return layers[w.get("index", 0)]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def tf32_peak_tflops():
    """Dense TF32 peak = measured bf16 peak x the nominal tf32/bf16 ratio (1/2)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["bf16_tflops"]) / 2, "measured bf16 burst x 0.5"
    return 1590.0 / 2, "fallback bf16 x 0.5"


# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the layer's kernel, from an ncu capture of exactly
# this launch (`--profile N` runs the bench's kernel on the bench's tensors); key: workload, plan variant. DRAM counters
# cannot be read outside a profiler, so the line carries these captured figures (null where none was taken).
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("mbv1_pw512", 36): 13936896 + 0,            # the 12.8 MB output is still in L2 when the kernel ends
    ("sweep_nb4_p70", 36): 99645440 + 35270656,  # stacked tiles of 512 rows
    ("mbv1_L1", 50): 102844672 + 148400128,
    ("mbv1_L7", 36): 26784768 + 63488,
    ("r50_3x3", 64): 15389696 + 131840,
    ("r50_3x3", 44): 15257344 + 1280,            # the per-tap kernel
    ("mbv1_pw512", 32): 14984448 + 256,
    ("sweep_nb4_p70", 32): 124626432 + 48126208,
    ("r50_3x3", 40): 17614080 + 0,
    ("sweep_nb4_p90", 14): 70554368 + 23536640,
}


def compulsory_bytes(L) -> int:
    """Activations read once + outputs written once + packed weights/indices + bias."""
    x = L.C * (L.Nc_out if L.R == 1 else L.Nc) * 4       # a strided 1x1 reads only the pixels it keeps
    y = L.M * L.Nc_out * 4
    w = L.m * L.Nb * L.R * 4 + L.m * 4 + (L.M + 1) * 4 + (L.M * 4 if L.bias is not None else 0)
    return x + y + w


class ClockSampler:
    """nvidia-smi clock / throttle-reason sampling during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "samples": len(sm),
                "reasons": sorted(reasons)}


def build_runner(ubp, torch, L, variant):
    """Returns (plan, run(stream-less call), pack_ms, plan_ms, device tensors)."""
    t0 = time.perf_counter()
    kmajor = L.name in KMAJOR_WORKLOADS
    if kmajor:
        blob = ubp.ubp_pack_kmajor(L.W[:, :, 0], L.mask, KMAJOR_B)
    else:
        blob = ubp.ubp_pack(L.W, L.mask, L.Nb)
    t1 = time.perf_counter()
    plan = ubp.Plan(blob, variant, kmajor=kmajor)
    torch.cuda.synchronize()
    t2 = time.perf_counter()
    X = torch.from_numpy(L.X).cuda()
    bias = torch.from_numpy(L.bias).cuda() if L.bias is not None else None
    if L.R == 9:
        Y = torch.empty((L.M, L.B, L.H, L.Wd), dtype=torch.float32, device="cuda")
        run = lambda: ubp.ubp_conv3x3_implicit(plan, X, bias, L.relu, out=Y)
    elif L.X.ndim == 4:
        Y = torch.empty((L.M, L.B, L.H, L.Wd), dtype=torch.float32, device="cuda")
        run = lambda: ubp.ubp_conv1x1(plan, X, bias, L.relu, out=Y)
    else:
        Y = torch.empty((L.M, L.Nc), dtype=torch.float32, device="cuda")
        run = lambda: ubp.ubp_spmm(plan, X, bias, L.relu, out=Y)
    return plan, run, (t1 - t0) * 1e3, (t2 - t1) * 1e3, X, Y, bias


def time_steps(torch, run, steps, warmup, flush_buf):
    """Per-step device times (ms) with CUDA events on the current stream; L2 flushed before every step."""
    for _ in range(warmup):
        if flush_buf is not None:
            flush_buf.zero_()
        run()
    torch.cuda.synchronize()
    evs = []
    for _ in range(steps):
        if flush_buf is not None:
            flush_buf.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); run(); b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


L2_BYTES = 126 * 1024 * 1024


def rotating_sets(torch, ubp, plan, L, X, bias, min_bytes=int(2.5 * L2_BYTES), max_sets=24):
    """Independent copies of the layer's activations, each with its own output tensor: as many as it takes for the
    set of all of them to exceed the L2 cache 2.5 times over (at least two), so that a step that walks through them
    in turn never finds its inputs or its output lines in L2. Returns (runs, tensors): runs[i]() launches the layer
    on copy i."""
    per_set = X.numel() * 4 + L.M * L.Nc * 4
    nsets = int(max(2, min(max_sets, -(-min_bytes // per_set))))
    runs, keep = [], []
    for i in range(nsets):
        Xi = X if i == 0 else X.clone()
        if L.R == 9:
            Yi = torch.empty((L.M, L.B, L.H, L.Wd), dtype=torch.float32, device="cuda")
            runs.append(lambda Xi=Xi, Yi=Yi: ubp.ubp_conv3x3_implicit(plan, Xi, bias, L.relu, out=Yi))
        elif L.X.ndim == 4:
            Yi = torch.empty((L.M, L.B, L.H, L.Wd), dtype=torch.float32, device="cuda")
            runs.append(lambda Xi=Xi, Yi=Yi: ubp.ubp_conv1x1(plan, Xi, bias, L.relu, out=Yi))
        else:
            Yi = torch.empty((L.M, L.Nc), dtype=torch.float32, device="cuda")
            runs.append(lambda Xi=Xi, Yi=Yi: ubp.ubp_spmm(plan, Xi, bias, L.relu, out=Yi))
        keep.append((Xi, Yi))
    return runs, keep


def time_region(torch, runs, steps, warmup, extra_regions=0, hold_s=0.0):
    """EXACTLY `steps` steps timed as ONE region: step i launches runs[i % len(runs)] (independent batches whose
    tensors together exceed L2, so every step starts cold), all of them enqueued from one CUDA graph on one stream
    and bracketed by one pair of CUDA events with a synchronize on both sides. Returns [ms of the region, ms of
    `extra_regions` repetitions...]; afterwards the same graph keeps replaying for `hold_s` seconds (untimed) so
    that a clock sampler sees the load. A pair of events around a single launch reads about 6 us even for an empty
    kernel on this hardware; bracketing the whole region, as a serving loop would run it, leaves that out and lets
    a launch start while its predecessor drains."""
    for i in range(warmup):
        runs[i % len(runs)]()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=torch.cuda.Stream()):
        for i in range(steps):
            runs[i % len(runs)]()
    graph.replay()                       # untimed: uploads the graph and counts as further warm-up
    torch.cuda.synchronize()
    out = []
    for _ in range(1 + extra_regions):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); graph.replay(); b.record()
        torch.cuda.synchronize()
        out.append(a.elapsed_time(b))
    t_end = time.perf_counter() + hold_s
    while time.perf_counter() < t_end:
        graph.replay()
        torch.cuda.synchronize()
    return out


def time_e2e(torch, ubp, plan, L, steps, warmup, nlanes=2):
    """Same step through the public call with HOST buffers: pinned X -> device, kernel, Y -> pinned host, every
    step. Steps alternate between two streams with their own device and host buffers, so that the upload of step
    i + 1 runs under the download of step i (PCIe is full duplex); the value is the steady-state rate."""
    bias = torch.from_numpy(L.bias).cuda() if L.bias is not None else None
    shape = (L.M, L.B, L.H, L.Wd) if L.X.ndim == 4 else (L.M, L.Nc)
    lanes = []
    for _ in range(nlanes):
        Xh = torch.from_numpy(L.X).pin_memory()
        lanes.append(dict(stream=torch.cuda.Stream(), Xh=Xh, Xd=torch.empty_like(Xh, device="cuda"),
                          Yd=torch.empty(shape, dtype=torch.float32, device="cuda"),
                          Yh=torch.empty(shape, dtype=torch.float32).pin_memory()))

    def step(i):
        ln = lanes[i % nlanes]
        with torch.cuda.stream(ln["stream"]):
            ln["Xd"].copy_(ln["Xh"], non_blocking=True)
            if L.R == 9:
                ubp.ubp_conv3x3_implicit(plan, ln["Xd"], bias, L.relu, out=ln["Yd"])
            elif L.X.ndim == 4:
                ubp.ubp_conv1x1(plan, ln["Xd"], bias, L.relu, out=ln["Yd"])
            else:
                ubp.ubp_spmm(plan, ln["Xd"], bias, L.relu, out=ln["Yd"])
            ln["Yh"].copy_(ln["Yd"], non_blocking=True)

    for i in range(max(warmup, nlanes)):
        step(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    cur = torch.cuda.current_stream()
    a.record(cur)
    for ln in lanes:
        ln["stream"].wait_event(a)
    for i in range(steps):
        step(i)
    for ln in lanes:
        cur.wait_stream(ln["stream"])
    b.record(cur)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps, lanes[0]["Xh"].numel() * 4, lanes[0]["Yh"].numel() * 4


def oracle_sample(L):
    """The bounded sample of the workload the oracle is run on: (activations of the sample, columns, description,
    callable that evaluates the oracle on it and returns (Yref, A) as [M][columns] arrays)."""
    import oracle
    dense_macs_per_col = L.M * L.C * L.R
    # aim at ~1 GMAC per call, at least 64 columns (3x3: whole images)
    if L.R == 9:
        nb = max(1, min(L.B, int(1.0e9 // (dense_macs_per_col * L.H * L.Wd * 0.2 + 1))))
        Xs = np.ascontiguousarray(L.X[:, :nb])
        cols = nb * L.H * L.Wd

        def fn():
            y, a = oracle.masked_conv3x3(L.W, L.mask, Xs, L.bias, relu=L.relu)
            return y.reshape(L.M, -1), a.reshape(L.M, -1)
        return Xs, cols, f"first {nb} of {L.B} images", fn
    X2 = L.X.reshape(L.C, -1)
    cols = int(max(64, min(X2.shape[1], 1.5e9 // dense_macs_per_col)))
    Xs = np.ascontiguousarray(X2[:, :cols])
    return Xs, cols, f"first {cols} of {X2.shape[1]} columns", lambda: oracle.masked_matmul(L.W, L.mask, Xs, L.bias, relu=L.relu)


def cpu_oracle_time(L, budget_s=20.0):
    """The oracle as it stands on the host cores, on a bounded sample of the workload's columns. Returns (effective
    GFLOP/s, threads, sample description, seconds per call, (Yref, A) of the sample)."""
    import oracle
    _, cols, sample, fn = oracle_sample(L)
    ref = fn()
    ts = []
    t_start = time.perf_counter()
    while len(ts) < 3 and time.perf_counter() - t_start < budget_s:
        t0 = time.perf_counter(); fn(); ts.append(time.perf_counter() - t0)
    t = float(np.median(ts))
    flops = 2.0 * L.m * L.Nb * L.R * cols
    return flops / t / 1e9, oracle.num_threads(), sample, t, ref


def error_figures(Y, Yref, A):
    """The three error figures of a result against the oracle's double-precision result on the same columns:
    scaled      max |Y - Yref| / (|Wm||X| + |bias|)           -- the gate (<= 1e-4)
    normwise    max |Y - Yref| / max |Yref|
    elementwise max |Y - Yref| / |Yref| over the outputs with |Yref| >= 1e-3 * rms(Yref)"""
    Y = np.asarray(Y, dtype=np.float64)
    d = np.abs(Y - Yref)
    scale = np.where(A > 0, A, 1.0)
    rms = float(np.sqrt(np.mean(Yref * Yref)))
    big = np.abs(Yref) >= 1e-3 * rms
    return {"scaled": float(np.max(d / scale)), "normwise": float(d.max() / max(float(np.abs(Yref).max()), 1e-300)),
            "elementwise": float(np.max(d[big] / np.abs(Yref[big]))) if big.any() else 0.0,
            "outputs_compared": int(Y.size)}


def roofline_us(L, hbm_gbs):
    """(time at the FP32 peak, time at the HBM copy bandwidth) of one layer, in microseconds."""
    return (2.0 * L.surviving_macs / (FP32_PEAK_TFLOPS * 1e12) * 1e6, compulsory_bytes(L) / (hbm_gbs * 1e9) * 1e6)


KERNEL_NAMES = ("ubp_spmm_kernel (sparse, FP32 FMA)", "ubp_tc_kernel (dense 3xTF32 on tcgen05, one CTA per tile)",
                "ubp_tc2_kernel (dense 3xTF32 on tcgen05, CTA pair per tile)",
                "ubp_tc3_kernel (dense 3xBF16 on tcgen05, CTA pair per tile)",
                "ubp_wros_kernel (the paper's loop over the canonical arrays, weight rotation, FP32 FMA)",
                "ubp_wros_kernel (the paper's loop over the canonical arrays, naive shift, FP32 FMA)",
                "ubp_conv3_kernel (3x3 on the padded pixel grid, taps as operand shifts, dense 3xBF16 on tcgen05, CTA pair per tile)",
                "ubp_tc3_kernel (dense 6xBF16 in three pieces on tcgen05, CTA pair per tile)")
ARITHMETIC = ("fp32 FMA, fp32 accumulate",
              "3 TF32 products per fp32 product, fp32 accumulate (error <= 2^-18 |w||x|)",
              "3 TF32 products per fp32 product, fp32 accumulate (error <= 2^-18 |w||x|)",
              "3 bf16 products per fp32 product, fp32 accumulate (error <= 3 * 2^-16 |w||x|)",
              "fp32 FMA, fp32 accumulate", "fp32 FMA, fp32 accumulate",
              "3 bf16 products per fp32 product, fp32 accumulate (error <= 3 * 2^-16 |w||x|)",
              "6 bf16 products of three exact pieces per fp32 product, fp32 accumulate (product error < 2^-23 |w||x|)")


def kernel_info(plan, L):
    """(index into KERNEL_NAMES / ARITHMETIC, [tile rows, tile columns]) of a fast-path launch of this plan."""
    if L.R == 9:
        kern, tile_rows, tile_cols = plan.tile_choice_conv(L.B, L.H, L.Wd, L.stride)
        if kern == 4:
            return 6, [tile_rows, tile_cols]
    else:
        kern, tile_rows, tile_cols = plan.tile_choice(L.Nc, 0)
    bf16 = 34 <= plan.variant <= 37 or 44 <= plan.variant <= 47 or 64 <= plan.variant <= 67
    if 84 <= plan.variant <= 87:
        return 7, [tile_rows, tile_cols]
    if L.R == 9 and plan.variant < 40:
        return 0, [tile_rows, tile_cols]
    if plan.variant in (60, 61):
        return plan.variant - 56, [tile_rows, tile_cols]
    if 70 <= plan.variant <= 73:
        return 0, [tile_rows, tile_cols]
    return (3 if (kern == 2 and bf16) else kern), [tile_rows, tile_cols]


def layer_roofline(L, us, hbm_gbs):
    """Roofline of one layer at `us` microseconds per launch: the slower of kept FLOPs at the FP32 peak and compulsory
    bytes at the measured copy bandwidth."""
    t_alu, t_hbm = roofline_us(L, hbm_gbs)
    return {"bound": "alu" if t_alu >= t_hbm else "hbm", "roofline_us": max(t_alu, t_hbm), "frac": max(t_alu, t_hbm) / us}


def measure_layer(ubp, torch, L, variant, steps, warmup, flush, hbm_gbs, name=None):
    """Plan + timed launches of one layer, same protocol as the headline: one region of `steps` launches over rotating
    batches (time_region); beside it the older per-step figure (a pair of events around every launch, L2 flushed by a
    256 MiB write before it). Returns (record, plan, Y): record = {workload, variant, kernel, arithmetic, tile, us
    (region time / steps), bound, roofline_us, frac, us_flushed (mean), frac_flushed}."""
    plan, run, pack_ms, plan_ms, X, Y, bias = build_runner(ubp, torch, L, variant)
    runs, keep = rotating_sets(torch, ubp, plan, L, X, bias)
    regions = time_region(torch, runs, steps, warmup, extra_regions=2)
    times = time_steps(torch, run, max(5, steps // 3), 3, flush)
    plan.check()
    us = regions[0] / steps * 1e3
    usf = float(np.mean(times)) * 1e3
    k, tile = kernel_info(plan, L)
    rec = {"workload": name or L.name, "M": L.M, "K": L.C * L.R, "Nc": L.Nc, "block": f"{L.Nb}x1x{L.R}",
           "sparsity_pct": L.sparsity_pct, "variant": plan.variant, "kernel": KERNEL_NAMES[k].split(" ")[0],
           "arithmetic": ARITHMETIC[k].split(",")[0], "tile": tile, "us": us,
           "us_regions": [r / steps * 1e3 for r in regions], "batches": len(runs),
           "eff_tflops": 2.0 * L.surviving_macs / us / 1e6}
    rec.update(layer_roofline(L, us, hbm_gbs))
    rec["us_flushed"] = usf
    rec["frac_flushed"] = rec["roofline_us"] / usf
    del runs, keep
    return rec, plan, Y


def workload_config(L, name, world, no_flush):
    """The `config` object of the JSON line: the workload and the measurement protocol (the same in both arms)."""
    return {"workload": name, "M": L.M, "K": L.C * L.R, "Nc": L.Nc, "block": f"{L.Nb}x1x{L.R}",
            "sparsity_pct": L.sparsity_pct, "blocks": L.m, "bias": L.bias is not None, "relu": bool(L.relu),
            "l2": "warm: one batch reused" if no_flush else
                  "cold: steps walk through independent batches whose tensors exceed L2 2.5 times over",
            "timed_region": "all steps enqueued from one CUDA graph, one event pair around them",
            "parallelism": f"replicated weights, columns sharded x{world}"}


# The other BASELINE configurations the default run measures beside the headline (every frac from the mean time)
EXTRA_CONFIGS = ["r50_3x3", "sweep_nb2_p50", "sweep_nb16_p50", "sweep_nb4_p70", "sweep_nb2_p90", "sweep_nb16_p90",
                 "sweep_nb4_p95"] + \
                [f"mbv1_L{i + 1}" for i in range(13)]
# The headline layer through the other arithmetics: three bf16 pieces (six products), TF32 products, fp32 FMA on the CUDA cores
HEADLINE_VARIANTS = [86, 32, 14]


def build_chained(ubp, torch, layers, variant):
    """Runners for layers that feed one another: a layer reads the output tensor of layer L.src (the block input for
    -1; by default its predecessor); strided layers produce the smaller planes."""
    plans, runs, keep, outs = [], [], [], []
    x0 = torch.from_numpy(layers[0].X).cuda()
    for li, L in enumerate(layers):
        src = li - 1 if L.src is None else L.src
        x = x0 if src < 0 else outs[src]
        plan = ubp.Plan(ubp.ubp_pack(L.W, L.mask, L.Nb), variant)
        bias = torch.from_numpy(L.bias).cuda() if L.bias is not None else None
        Ho, Wo = (L.H - 1) // L.stride + 1, (L.Wd - 1) // L.stride + 1
        y = torch.empty((L.M, L.B, Ho, Wo), dtype=torch.float32, device="cuda")
        fn = ubp.ubp_conv3x3_implicit if L.R == 9 else ubp.ubp_conv1x1
        kw = {}
        if L.stride != 1:
            kw["stride"] = L.stride
            if L.R == 1:
                kw["scratch"] = torch.empty(L.C * L.B * Ho * Wo, dtype=torch.float32, device="cuda")
            else:       # stride-2 3x3: the phase planes (allocated here so that the launches can be captured in a graph)
                need = ubp.load().ubp_conv3x3_strided_scratch(L.C, L.B, L.H, L.Wd, L.stride)
                if need:
                    kw["scratch"] = torch.empty(need // 4, dtype=torch.float32, device="cuda")
        runs.append(lambda fn=fn, plan=plan, x=x, bias=bias, relu=L.relu, y=y, kw=kw: fn(plan, x, bias, relu, out=y, **kw))
        plans.append(plan); keep.append((x, y, bias, kw)); outs.append(y)
    return plans, runs, keep


def run_chain(args, torch, ubp, rank, world, dist, cfg="mbv1_chain"):
    """mbv1_chain: the 13 pointwise layers of the MobileNetV1-shaped network (batch 64, 1x4 blocks, 80 %, bias+ReLU,
    independent seeded inputs per layer). r50_bottleneck: a ResNet-50-shaped bottleneck (1x1, 3x3, 1x1; batch 32,
    blocks of 4, 80 %), each layer reading its predecessor's output. One step = all launches replayed from one
    CUDA graph."""
    layers = ubp_synth.config_layers(cfg, index=rank)
    hbm_gbs, peak_src = measured_peaks()
    runs, plans, keep = [], [], []
    if cfg in ("r50_bottleneck", "r50_downsample"):
        plans, runs, keep = build_chained(ubp, torch, layers, args.variant)
    else:
        for L in layers:
            plan, run, _, _, X, Y, bias = build_runner(ubp, torch, L, args.variant)
            plans.append(plan); runs.append(run); keep.append((X, Y, bias))
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")

    def one_pass():
        for run in runs:
            run()
    one_pass()                  # warm every kernel outside the capture (first-launch attribute set-up)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    cap_stream = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=cap_stream):
        one_pass()
    per_layer = []
    for L, run in zip(layers, runs):
        ts = time_steps(torch, run, max(5, args.steps // 5), 3, flush)
        per_layer.append(float(np.median(ts)) * 1e3)
    flushed = time_steps(torch, graph.replay, max(5, args.steps // 3), 3, flush)
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    # the timed region: `steps` passes over the chain, all launches from one CUDA graph, one event pair around them
    regions = time_region(torch, [one_pass], args.steps, args.warmup, extra_regions=1, hold_s=0.4)
    clocks = sampler.stop()
    times = [regions[0] / args.steps]
    for p in plans:
        p.check()
    step_ms = max_over_ranks(float(np.mean(times)), dist, torch, "cuda")
    flops = sum(2.0 * L.surviving_macs for L in layers)
    roofs = [roofline_us(L, hbm_gbs) for L in layers]
    roof_total_us = sum(max(r) for r in roofs)
    line = {
        "metric": f"effective GFLOP/s (2 x surviving MACs / time) of the {len(layers)}-layer chain",
        "value": aggregate_gflops(flops, world, step_ms), "unit": "GFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 in/out/accumulate; per layer fp32 FMA or bf16x3 products (layers[].variant)",
        "data": "synthetic",
        "config": {"workload": cfg, "layers": len(layers), "batch": layers[0].B, "block": "4x1xR", "sparsity_pct": 80,
                   "launch": f"{len(layers)} kernels per step; all steps replayed from one CUDA graph, one event pair around them",
                   "l2": "not flushed: the chain's tensors (about 1.5 GB) exceed L2 many times over" if cfg == "mbv1_chain"
                         else "not flushed: the three layers' tensors (about 70 MB) partly stay in L2 from step to step"},
        "per_step_flushed": {"us_mean": float(np.mean(flushed)) * 1e3, "frac": roof_total_us / (float(np.mean(flushed)) * 1e3),
                             "protocol": "one graph replay of the chain per event pair, L2 flushed by a 256 MiB write before it"},
        "roofline": {"bound": "mixed (per layer: see layers)", "roofline_us": roof_total_us,
                     "frac_of_roofline_time": roof_total_us / (step_ms * 1e3),
                     "peak_source": f"FP32 74.45 TFLOP/s derived; HBM {hbm_gbs} GB/s {peak_src}"},
        "layers": [{"name": L.name, "M": L.M, "K": L.C * L.R, "Nc": L.Nc_out, "stride": L.stride, "variant": p.variant, "us_flushed": us,
                    "roofline_us": max(r), "bound": "alu" if r[0] >= r[1] else "hbm", "frac_flushed": max(r) / us}
                   for L, p, us, r in zip(layers, plans, per_layer, roofs)],
        "clocks": clocks, "gpu_launches": len(layers) * args.steps,
    }
    if rank == 0:
        print(json.dumps(line), flush=True)


# Per-layer comparison of pruning patterns and dataflows (the paper's Section 5.4 on B200): layer shape, sparsity
CMP_WORKLOADS = {
    "cmp_pw512_p80": dict(M=512, C=512, B=64, H=14, Wd=14, p=80, w_scale=0.05),
    "cmp_pw512_p90": dict(M=512, C=512, B=64, H=14, Wd=14, p=90, w_scale=0.05),
    "cmp_2048_p80": dict(M=2048, C=2048, Nc=8192, p=80, w_scale=0.02),
    "cmp_2048_p90": dict(M=2048, C=2048, Nc=8192, p=90, w_scale=0.02),
}
CMP_PATTERNS = [("EP", 1, False), ("ABP 1x2", 2, True), ("UBP 1x2", 2, False), ("ABP 1x4", 4, True), ("UBP 1x4", 4, False)]
CMP_KERNELS = [("plan, sparse FP32 kernel", {1: 17, 2: 15, 4: 14}), ("paper loop, weight rotation (60)", 60),
               ("paper loop, naive shift (61)", 61), ("plan, tensor-core bf16x3 kernel", {1: 34, 2: 35, 4: 36})]


def cmp_layer(name, pattern_index, seed_index=0):
    w = CMP_WORKLOADS[name]
    label, nb, aligned = CMP_PATTERNS[pattern_index]
    kw = dict(Nc=w["Nc"], x_dist="normal") if "Nc" in w else dict(B=w["B"], H=w["H"], Wd=w["Wd"])
    return ubp_synth.make_layer(f"{name}:{label}", w["M"], w["C"], nb, w["p"], 8000 + 10 * seed_index + pattern_index,
                                w_scale=w["w_scale"], aligned=aligned, **kw)


def run_cmp(args, name, rank, local_rank, world):
    """Element-wise, aligned and unaligned pruning of one layer at one sparsity through (a) the plan-based sparse
    kernel, (b) the two kernels that keep the paper's own loop over the canonical arrays, with weight rotation and
    naive, (c) the tensor-core kernel. One JSON line; `comparison` holds the table (us per launch, region protocol)
    and the ratios Section 5.4 discusses: unaligned / aligned and naive / weight-rotating."""
    import torch
    import paper_2407_19644_b200 as ubp
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    ubp.load()
    torch.cuda.set_device(local_rank)
    hbm_gbs, _ = measured_peaks()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    steps = max(10, min(args.steps, 40))
    table = {}
    head = None
    sampler = ClockSampler(local_rank)
    sampler.start()
    for pi, (label, nb, aligned) in enumerate(CMP_PATTERNS):
        L = cmp_layer(name, pi, seed_index=rank)
        row = {}
        for kname, v in CMP_KERNELS:
            variant = v[nb] if isinstance(v, dict) else v
            rec, plan, Y = measure_layer(ubp, torch, L, variant, steps, 3, flush, hbm_gbs, name=f"{name}:{label}")
            row[kname] = {"us": rec["us"], "us_flushed": rec["us_flushed"], "variant": rec["variant"], "frac": rec["frac"]}
            if label == "UBP 1x4" and variant == 14:
                head = (L, rec)
            del plan, Y
            torch.cuda.empty_cache()
        table[label] = row
    clocks = sampler.stop()
    ratios = {}
    for kname, _ in CMP_KERNELS[:3]:
        ratios[kname] = {f"UBP/ABP 1x{nb}": table[f"UBP 1x{nb}"][kname]["us"] / table[f"ABP 1x{nb}"][kname]["us"] for nb in (2, 4)}
        ratios[kname].update({f"EP/UBP 1x{nb}": table["EP"][kname]["us"] / table[f"UBP 1x{nb}"][kname]["us"] for nb in (2, 4)})
    ratios["naive/weight-rotating"] = {lab: table[lab][CMP_KERNELS[2][0]]["us"] / table[lab][CMP_KERNELS[1][0]]["us"]
                                       for lab in ("UBP 1x2", "UBP 1x4", "ABP 1x2", "ABP 1x4")}
    L, rec = head
    line = {"metric": METRIC, "value": 2.0 * L.surviving_macs / rec["us"] / 1e3, "unit": "GFLOP/s", "n_gpus": 1,
            "steps": steps, "warmup": 3, "ms_per_step": rec["us"] / 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(L, name, 1, False), headline_cell="UBP 1x4 through the plan-based sparse kernel"),
            "roofline": {"bound": rec["bound"], "frac": rec["frac"], "roofline_us": rec["roofline_us"]},
            "comparison": {"us_per_launch": table, "ratios": ratios,
                           "paper": "Section 5.4 (phone CPU): unaligned with weight rotation about equal to aligned, the "
                                    "naive unaligned kernel clearly slower, larger blocks faster than element-wise"},
            "clocks": clocks, "gpu_launches": steps}
    if rank == 0:
        print(json.dumps(line), flush=True)


def max_over_ranks(ms: float, dist, torch, device) -> float:
    """A step is as slow as its slowest rank: MAX-reduce the per-rank device time (no-op without a group)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gflops(flops_per_rank: float, world: int, step_ms: float) -> float:
    """Whole-job throughput: every rank does the same amount of work on its own columns (weak scaling)."""
    return world * flops_per_rank / (step_ms * 1e-3) / 1e9


def run_reference(args, L, name):
    """--impl reference: the CPU oracle timed on this machine's host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    vals = []
    sample = ""
    for i in range(args.warmup + args.steps):
        g, cores, sample, t, _ = cpu_oracle_time(L, budget_s=1.0)
        if i >= args.warmup:
            vals.append((g, t))
        if i >= args.warmup + 2 and sum(t for _, t in vals) > 90:
            break
    g = float(np.median([v for v, _ in vals]))
    t = float(np.median([t for _, t in vals]))
    line = {"metric": METRIC, "value": g, "unit": "GFLOP/s",
            "impl": "reference", "n_gpus": args.gpus, "steps": len(vals), "warmup": args.warmup,
            "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(L, name, args.gpus, args.no_flush),
            "cpu_baseline": {"value": g, "unit": "GFLOP/s", "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": g, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def cpu_bed_time(W, Nb: int, m: int, budget_s: float = 15.0):
    """Time of the sequential oracle (scores, Algorithm 1, Algorithm 2) for this layer on the host. Algorithm 1 is run
    for a bounded number of its m iterations (each costs the same arg max over the remaining score list) and scaled."""
    import oracle
    t0 = time.perf_counter()
    S = oracle.block_scores(W, Nb)
    t_scores = time.perf_counter() - t0
    n = min(m, 64)
    t0 = time.perf_counter()
    oracle.bed_expand(S, Nb, n)
    t_n = time.perf_counter() - t0
    n2 = int(min(m, max(n, budget_s / max(t_n / max(n, 1), 1e-9))))
    t0 = time.perf_counter()
    Ibar, _ = oracle.bed_expand(S, Nb, n2)
    t_exp = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle.bed_divide(Ibar, Nb)
    t_div = time.perf_counter() - t0
    full = t_scores + (t_exp + t_div) * (m / max(n2, 1))
    sample = (f"scores of the whole layer + first {n2} of {m} iterations of Algorithm 1 on the full score list "
              f"(then Algorithm 2), scaled by {m / max(n2, 1):.2f}" if n2 < m else "the whole selection")
    return full, 1, sample


def run_bed(args, name, rank, local_rank, world):
    """One step = one block selection (scores, expansion, threshold, mask) of the layer's dense weights resident in
    HBM. Every rank selects for its own layer of the same shape (layers are independent: no collective)."""
    M, C, R, Nb, p = BED_WORKLOADS[name]
    W = ubp_synth.selection_weights(M, C, R, seed=9000 + rank, kind="trained")
    m = ubp_synth.block_budget(M, C, p, Nb)
    metric = "blocks selected per second by block expansion and division (m / time)"
    cfg = {"workload": name, "M": M, "C": C, "R": R, "block": f"{Nb}x1x{R}", "sparsity_pct": p, "blocks": m,
           "candidates": M * C}
    if args.impl == "reference":
        if rank != 0:
            return
        import oracle
        vals = []
        for i in range(args.warmup + args.steps):
            t, cores, sample = cpu_bed_time(W, Nb, m, budget_s=2.0)
            if i >= args.warmup:
                vals.append(t)
            if i >= args.warmup + 2 and sum(vals) > 0 and (i + 1) * 3.0 > 120:
                break
        t = float(np.median(vals))
        cfg["sample"] = sample
        print(json.dumps({"metric": metric, "value": m / t, "unit": "blocks/s", "impl": "reference", "n_gpus": args.gpus,
                          "steps": len(vals), "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
                          "cpu_baseline": {"value": m / t, "unit": "blocks/s", "cores": cores, "kind": "oracle", "sample": sample},
                          "e2e": {"value": m / t, "unit": "blocks/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}),
              flush=True)
        return
    import torch
    import paper_2407_19644_b200 as ubp
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    ubp.load()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sel = ubp.BedSelector(M, C, R, Nb)
    Wd = torch.from_numpy(W).cuda()
    mask = torch.empty((M, C), dtype=torch.uint8, device="cuda")
    nsel = torch.zeros(1, dtype=torch.int64, device="cuda")
    run = lambda: sel.select(Wd, m, mask, nsel)          # noqa: E731
    if args.profile > 0:
        for _ in range(args.profile):
            run()
        torch.cuda.synchronize()
        print(json.dumps({"profile_launches": args.profile, "workload": name, "selected": int(nsel.item())}), flush=True)
        return
    flush = None if args.no_flush else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    times = time_steps(torch, run, args.steps, args.warmup, flush)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if int(nsel.item()) != m:
        raise SystemExit(f"selected {int(nsel.item())} blocks, wanted {m}")
    step_ms = max_over_ranks(float(np.mean(times)), dist, torch, "cuda")
    # the same nine launches replayed from one CUDA graph (the calls only enqueue work, so they can be captured)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=torch.cuda.Stream()):
        run()
    graph_ms = float(np.mean(time_steps(torch, graph.replay, max(5, args.steps // 2), 3, flush)))
    if int(nsel.item()) != m:
        raise SystemExit(f"graph replay selected {int(nsel.item())} blocks, wanted {m}")
    # end to end: weights from pinned host memory, mask back to pinned host memory
    Wh = torch.from_numpy(W).pin_memory()
    mh = torch.empty((M, C), dtype=torch.uint8).pin_memory()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    et = []
    for i in range(3 + max(5, min(args.steps, 20))):
        torch.cuda.synchronize()
        e0.record()
        Wd.copy_(Wh, non_blocking=True)
        run()
        mh.copy_(mask, non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            et.append(e0.elapsed_time(e1))
    e2e_ms = max_over_ranks(float(np.mean(et)), dist, torch, "cuda")
    line = {
        "metric": metric, "value": world * m / (step_ms * 1e-3), "unit": "blocks/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "us_min": float(np.min(times)) * 1e3,
        "us_median": float(np.median(times)) * 1e3, "graph_replay_ms_per_step": graph_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": dict(cfg, l2="warm" if args.no_flush else "flushed between steps (256 MiB write)",
                       parallelism=f"independent layers x{world}"),
        "roofline": {"bound": "latency", "achieved": None, "peak": None, "unit": None, "frac": None, "traffic": None,
                     "note": "a chain of dependent arg max / re-score rounds per input channel (at most M/Nb of them); "
                             "neither memory traffic nor arithmetic is near a hardware limit",
                     "candidates_per_second": M * C / (step_ms * 1e-3)},
        "clocks": clocks, "gpu_launches": args.steps * 9,
        "e2e": {"value": world * m / (e2e_ms * 1e-3), "unit": "blocks/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": W.nbytes, "d2h_bytes_per_step": M * C},
    }
    if rank == 0 and not args.no_cpu:
        t, cores, sample = cpu_bed_time(W, Nb, m)
        line["cpu_baseline"] = {"value": m / t, "unit": "blocks/s", "cores": cores, "kind": "oracle", "sample": sample,
                                "seconds_for_the_layer": t}
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="mbv1_pw512")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--no-flush", action="store_true", help="do not flush L2 between steps (warm-L2 figure)")
    ap.add_argument("--headline-only", action="store_true",
                    help="default workload only: skip the other arithmetics and the other configurations")
    ap.add_argument("--profile", type=int, default=0, metavar="N",
                    help="build the plan, launch the layer N times and exit (a small target for ncu captures)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s): start bench.py with "
                         f"torch.distributed.run --nproc-per-node {args.gpus}, or with no launcher at all")
    name = args.workload
    if name in ("mbv1_chain", "r50_bottleneck", "r50_downsample"):
        if args.impl == "reference":
            raise SystemExit("--impl reference times single layers; pick a layer workload")
        import torch
        import paper_2407_19644_b200 as ubp
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
        ubp.load()
        torch.cuda.set_device(local_rank)
        dist = None
        if world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        run_chain(args, torch, ubp, rank, world, dist, cfg=name)
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    if name in BED_WORKLOADS:
        run_bed(args, name, rank, local_rank, world)
        return
    if name in CMP_WORKLOADS:
        if args.impl == "reference":
            raise SystemExit("--impl reference times single layers; pick a layer workload")
        run_cmp(args, name, rank, local_rank, world)
        return
    L = get_layer(name, seed_index=rank)

    if args.impl == "reference":
        run_reference(args, L, name)
        return

    import torch
    import paper_2407_19644_b200 as ubp
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    ubp.load()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    plan, run, pack_ms, plan_ms, X, Y, bias = build_runner(ubp, torch, L, args.variant)
    if args.profile > 0:
        for _ in range(args.profile):
            run()
        torch.cuda.synchronize()
        plan.check()
        print(json.dumps({"profile_launches": args.profile, "workload": name, "variant": plan.variant}), flush=True)
        return
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    runs, keep = ([run], []) if args.no_flush else rotating_sets(torch, ubp, plan, L, X, bias)

    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    regions = time_region(torch, runs, args.steps, args.warmup, extra_regions=2, hold_s=0.4)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["sampled"] = "from the timed region on, while the same graph kept replaying for 0.4 s"
    plan.check()
    launches = args.steps
    step_ms = max_over_ranks(regions[0] / args.steps, dist, torch, "cuda")
    # the older per-step protocol beside it: a pair of events around every launch, L2 flushed by a 256 MiB write
    times = time_steps(torch, run, max(10, min(args.steps, 50)), 3, flush)
    plan.check()
    del runs, keep
    e2e_ms, h2d, d2h = time_e2e(torch, ubp, plan, L, max(5, min(args.steps, 30)), 3)
    e2e_ms = max_over_ranks(e2e_ms, dist, torch, "cuda")

    flops = 2.0 * L.surviving_macs
    gflops = aggregate_gflops(flops, world, step_ms)
    hbm_gbs, peak_src = measured_peaks()
    t_alu = flops / (FP32_PEAK_TFLOPS * 1e12)
    t_hbm = compulsory_bytes(L) / (hbm_gbs * 1e9)
    per_gpu_tflops = flops / (step_ms * 1e-3) / 1e12
    if t_alu >= t_hbm:
        roof = {"bound": "alu", "achieved": per_gpu_tflops, "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s",
                "frac": per_gpu_tflops / FP32_PEAK_TFLOPS, "traffic": None,
                "peak_source": "148 SMs x 128 FP32 lanes x 2 x 1.965 GHz (derived)"}
    else:
        ach = compulsory_bytes(L) / (step_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s", "frac": ach / hbm_gbs,
                "traffic": None, "peak_source": f"{peak_src} copy bandwidth"}
    roof["roofline_us"] = max(t_alu, t_hbm) * 1e6
    roof["frac_of_roofline_time"] = max(t_alu, t_hbm) / (step_ms * 1e-3)
    roof["traffic"] = NCU_DRAM_BYTES_PER_LAUNCH.get((name, plan.variant))
    roof["algorithmic_bytes"] = compulsory_bytes(L)
    k, tile = kernel_info(plan, L)
    roof["kernel"] = KERNEL_NAMES[k]
    roof["arithmetic"] = ARITHMETIC[k]
    roof["tile"] = tile
    if plan.variant >= 30 and k > 0:
        # the tensor-core variants do 3 x the DENSE multiply-adds; report that rate against the tensor peak of the
        # operand type too (bf16: the measured cuBLAS figure; TF32: half of it, the nominal ratio)
        dense_tf = 3 * 2.0 * L.M * L.C * L.R * L.Nc / (step_ms * 1e-3) / 1e12
        tf32_peak = tf32_peak_tflops()
        if k == 3:
            roof["tensor"] = {"dense_bf16_tflops": dense_tf, "peak": tf32_peak[0] * 2,
                              "peak_source": tf32_peak[1].replace(" x 0.5", ""), "frac": dense_tf / (tf32_peak[0] * 2)}
        else:
            roof["tensor"] = {"dense_tf32_tflops": dense_tf, "peak": tf32_peak[0], "peak_source": tf32_peak[1],
                              "frac": dense_tf / tf32_peak[0]}

    dtype = "f32" if k == 0 else ("f32 in/out/accumulate; bf16x3 products" if k == 3 else "f32 in/out/accumulate; tf32x3 products")
    line = {
        "metric": METRIC, "value": gflops, "unit": "GFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
        "us_per_layer": step_ms * 1e3, "us_per_layer_regions": [r / args.steps * 1e3 for r in regions],
        "per_step_flushed": {"us_mean": float(np.mean(times)) * 1e3, "us_median": float(np.median(times)) * 1e3,
                             "us_min": float(np.min(times)) * 1e3, "steps": len(times),
                             "frac": max(t_alu, t_hbm) / (float(np.mean(times)) * 1e-3),
                             "protocol": "a pair of CUDA events around every launch, L2 flushed by a 256 MiB write before "
                                         "it; two events around an empty kernel read about 6 us here"},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
        "arithmetic": roof.get("arithmetic"),
        "config": workload_config(L, name, world, args.no_flush),
        "variant": plan.variant,
        "roofline": roof, "clocks": clocks,
        "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e9, "unit": "GFLOP/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "overlap": "steps alternate between two streams with their own buffers"},
        "offline": {"pack_ms": pack_ms, "plan_ms": plan_ms, "plan_bytes": plan.dev_bytes},
    }
    ref = None
    if rank == 0 and not args.no_cpu:
        g, cores, sample, _, ref = cpu_oracle_time(L)
        line["cpu_baseline"] = {"value": g, "unit": "GFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}
        # the oracle's outputs on that sample also give the error figures of what the timed kernel wrote
        run()
        torch.cuda.synchronize()
        ncol = ref[0].shape[1]
        line["errors"] = dict(error_figures(Y.reshape(L.M, -1)[:, :ncol].cpu().numpy(), *ref), sample=sample)
        launches += 1
    extras = rank == 0 and not args.headline_only and name == "mbv1_pw512" and args.variant == 0
    if extras:
        # the same layer, same protocol, through the other two arithmetics; error figures on the oracle's sample
        esteps = max(10, min(args.steps, 100))           # the headline's region length by default
        line["variants"] = []
        for v in HEADLINE_VARIANTS:
            rec, pv, Yv = measure_layer(ubp, torch, L, v, esteps, 3, flush, hbm_gbs, name=name)
            launches += esteps + 3
            if ref is not None:
                rec["errors"] = error_figures(Yv.reshape(L.M, -1)[:, :ref[0].shape[1]].cpu().numpy(), *ref)
            line["variants"].append(rec)
            del pv, Yv
        # the other BASELINE configurations (automatic variant), each timed like the headline
        del X, Y, plan, run
        line["configs"] = []
        for cname in EXTRA_CONFIGS:
            Lc = get_layer(cname, seed_index=rank)
            rec, pc, Yc = measure_layer(ubp, torch, Lc, 0, esteps, 3, flush, hbm_gbs, name=cname)
            launches += esteps + 3
            line["configs"].append(rec)
            del pc, Yc, Lc
            torch.cuda.empty_cache()
        chain = [r for r in line["configs"] if r["workload"].startswith("mbv1_L")]
        worst = min(line["configs"], key=lambda r: r["frac"])
        upto90 = [r for r in line["configs"] if r["sparsity_pct"] <= 90]
        line["configs_summary"] = {"min_frac": worst["frac"], "min_frac_workload": worst["workload"],
                                   "min_frac_up_to_90pct_sparsity": min(r["frac"] for r in upto90),
                                   "chain_us_sum": sum(r["us"] for r in chain),
                                   "chain_roofline_us_sum": sum(r["roofline_us"] for r in chain),
                                   "steps_each": esteps, "frac_from": "mean"}
    line["gpu_launches"] = args.steps                 # inside the timed region: one kernel per step
    line["gpu_launches_beside"] = launches - args.steps + len(times) + 3 * args.steps   # warm-up replay, two more regions,
                                                                                      # flushed steps, variants and configs
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def spawn_ranks(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start N local ranks of this script under torch.distributed.run
    (one per GPU, rendezvous on 127.0.0.1) and return their exit code. Rank 0 prints the line."""
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


if __name__ == "__main__":
    main()
