#!/usr/bin/env python
"""Benchmark of libgconv on B200: grouped-conv GFLOP/s and ms/layer vs groups, % of roofline.

One "step" = one pass of the hot path over the WideResNet-40-2-shaped stack (18 grouped 3x3
layers: 32/64/128 channels at 32/16/8, stride-2 transitions) at batch 128 for every group count in
{1,2,4,8,16}: 90 gconv_forward launches.  Every layer instance owns its x and y buffers, so ~1.8 GB
is cycled between two uses of the same buffer (more than the 126 MB L2).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--quick]

Prints ONE JSON line.  `value` is GFLOP/s (2*MACs of Eq. (2) of the paper per second) with inputs
resident in HBM, the step replayed as a CUDA graph; `e2e` is the same metric through
gconv_forward_host with pinned host buffers (copies inside the timed region).  The same line carries
the per-layer tables of every benchmark family (ms, GFLOP/s, GB/s, fraction of the layer's roofline,
cold and warm L2, the plain-copy and launch-interval floors beside them), the time-falls-with-groups
checks and a `targets` object that names every layer below the 50 % tensor / 60 % HBM bars.
`--impl reference` times the CPU oracle (the only reference there is: the paper ships no code) on
a bounded sample.
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

import numpy as np  # noqa: E402

from paper_2006_09791_b200 import synth, workloads as wl  # noqa: E402
from paper_2006_09791_b200.torch_util import attach_workspace  # noqa: E402

METRIC = "grouped_conv_gflops"
UNIT = "GFLOP/s"
WORKLOAD = "wrn40_2_stack_N128_groups_1_2_4_8_16"
BATCH = 128
CPU_SAMPLE_BATCH = 8      # batch of the reference arm's per-step sample
CPU_LEG_BATCH = 32        # batch of the cpu_baseline leg of the GPU arm
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes one launch of the dominant kernel moves on average over the step come from an ncu capture whose summary is
# kept under profiles/ (a table row per kernel variant: bytes per launch, the commit it was captured at, the command).
NCU_TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.md")


def ncu_traffic():
    """{variant name: {"bytes": DRAM bytes per launch, "commit": ..., "note": ...}} parsed from the committed table."""
    out = {}
    try:
        for ln in open(NCU_TRAFFIC_TABLE):
            f = [t.strip() for t in ln.strip().strip("|").split("|")]
            if len(f) >= 3 and f[0] and not f[0].startswith(("-", "kernel")):
                try:
                    out[f[0]] = {"bytes": float(f[1]), "commit": f[2], "note": f[3] if len(f) > 3 else ""}
                except ValueError:
                    pass
    except OSError:
        pass
    return out


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def step_layers(batch):
    """[(groups, Layer)] of one step, repeats expanded (90 entries at the full workload)."""
    out = []
    for g in wl.WRN_GROUPS:
        for L in wl.wrn_stack(g, batch):
            out.extend([(g, L)] * L.repeat)
    return out


# ------------------------------------------------------------------------------------------------
# clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
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
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm
def oracle_sample_time(batch, threads):
    """Runs the oracle as it stands over the stack at a reduced batch; returns (seconds, macs)."""
    import oracle
    total_macs, total_s = 0, 0.0
    cache = {}
    for g in wl.WRN_GROUPS:
        for L in wl.wrn_stack(g, batch):
            key = (L.C_in, L.H, L.C_out, g)
            if key not in cache:
                cache[key] = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, g, synth.layer_seed(1, *key))
            x, w = cache[key]
            t0 = time.perf_counter()
            for _ in range(L.repeat):
                oracle.gconv_ref(x, w, L.stride, L.pad, L.dilation, g, threads=threads)
            total_s += time.perf_counter() - t0
            total_macs += L.macs * L.repeat
    return total_s, total_macs


def gspc_baseline(threads, batch=CPU_SAMPLE_BATCH):
    """The paper's own method (Algorithm 1: kernels packed ahead of time, then input reshaping, convolution on the
    packed volumes and output reshaping, float32) timed on the host cores over the same stack at a reduced batch, for
    a few (T_I, T_O) tile pairs within Eq. (1)'s bounds: each pair is capped by CPG and KPG of the layer.  A second
    reported CPU baseline; not the oracle, not a target."""
    import oracle
    pairs = [(1, 1), (4, 8), (8, 16), (16, 16), (32, 32), (128, 128)]
    results = []
    for T_I, T_O in pairs:
        secs, macs, stages = 0.0, 0, [0.0, 0.0, 0.0]
        for g in wl.WRN_GROUPS:
            for L in wl.wrn_stack(g, batch):
                ti, to = min(T_I, L.Cg), min(T_O, L.Kg)
                x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, g, synth.layer_seed(1, L.C_in, L.H, L.C_out, g))
                wp = oracle.gspc_pack_kernels(w, g, ti, to)
                t0 = time.perf_counter()
                for _ in range(L.repeat):
                    _, st = oracle.gspc_forward(x, wp, w.shape, L.stride, L.pad, L.dilation, g, ti, to, threads=threads, return_stage_seconds=True)
                    stages = [a + b for a, b in zip(stages, st)]
                secs += time.perf_counter() - t0
                macs += L.macs * L.repeat
        results.append({"T_I": T_I, "T_O": T_O, "value": 2.0 * macs / secs / 1e9, "seconds": secs,
                        "stage_seconds": {"input_reshape": stages[0], "convolution": stages[1], "output_reshape": stages[2]}})
    best = max(results, key=lambda r: r["value"])
    return {"value": best["value"], "unit": UNIT, "cores": threads, "kind": "gspc_algorithm1_f32", "best_tiles": [best["T_I"], best["T_O"]],
            "tile_sweep": results,
            "sample": "the 18-layer stack at N=%d (of %d) for every group count; tiles capped by CPG and KPG per layer" % (batch, BATCH)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    threads = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
    sample = "the 18-layer stack at N=%d (of %d) for every group count, oracle as it stands" % (CPU_SAMPLE_BATCH, BATCH)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_time(1, threads)
    secs, macs = 0.0, 0
    for _ in range(args.steps):
        s, m = oracle_sample_time(CPU_SAMPLE_BATCH, threads)
        secs += s
        macs += m
    value = 2.0 * macs / secs / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# multi-rank helpers (replicas only: ranks share nothing but the clock)
def reduce_max_over_ranks(value, world, device=None):
    """Largest `value` over all ranks (the job is as slow as its slowest replica)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(flops_per_rank_step, world, ms_max):
    """Whole-job throughput in GFLOP/s: every replica does the same step, the clock is the slowest rank's."""
    return world * flops_per_rank_step / (ms_max * 1e-3) / 1e9


# ------------------------------------------------------------------------------------------------
# GPU arm
class Instance:
    """One layer instance of the step: descriptor, packed weights, its own x and y buffers."""

    def __init__(self, g, L, x_dev, wp, torch, gconv):
        self.g, self.L = g, L
        self.desc = gconv.gconv_desc_create(*L.desc_args())
        self.x = x_dev
        self.wp = wp
        self.y = torch.empty(L.y_elems, dtype=torch.float32, device=x_dev.device)
        self.ws = attach_workspace(self.desc, x_dev.device)


def time_layer(torch, gconv, L, stream, reps=160, min_cycle_bytes=2 * L2_BYTES + (64 << 20), warm=False):
    """Average device time of one gconv_forward launch of layer L with cold L2: launches rotate over
    enough distinct (x, y) buffer pairs that more than twice the L2 is cycled between reuses.  With `warm` the
    launches reuse ONE buffer pair instead (whatever fits stays in L2).  Returns (median ms, variant)."""
    if warm:
        min_cycle_bytes = 0
    dev = torch.device("cuda", torch.cuda.current_device())
    per = 4 * (L.x_elems + L.y_elems)
    nbuf = 1 if warm else max(2, -(-min_cycle_bytes // per))
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        ws = attach_workspace(d, dev)
        x0, w0 = synth.make_layer_tensors(min(L.N, 2), L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups, 99, L.x_dist)
        w = torch.from_numpy(w0).to(dev)
        reps_x = -(-L.N // x0.shape[0])
        xs = [torch.from_numpy(x0).to(dev).repeat(reps_x, 1, 1, 1)[:L.N].contiguous() for _ in range(nbuf)]
        ys = [torch.empty(L.y_elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        with torch.cuda.stream(stream):
            gconv.gconv_pack_weights(d, w, wp, stream)
            for i in range(min(nbuf, 5) + 3):
                gconv.gconv_forward(d, xs[i % nbuf], wp, ys[i % nbuf], stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph = torch.cuda.CUDAGraph()
            stream.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(reps):
                    gconv.gconv_forward(d, xs[i % nbuf], wp, ys[i % nbuf], stream)
            graph.replay()
            stream.synchronize()
            times = []
            for _ in range(5):
                e0.record(stream)
                graph.replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1) / reps)
        st = gconv.gconv_last_status(d, stream)
        assert st == 0, gconv.status_string(st)
        return statistics.median(times), gconv.gconv_variant(d)
    finally:
        gconv.gconv_desc_destroy(d)


def time_block(torch, gconv, L, C2, stream, reps=20, min_cycle_bytes=2 * L2_BYTES + (64 << 20)):
    """Average device time of one gconv_block_forward launch (grouped 3x3 of layer L, then pointwise C_out -> C2)
    with cold L2, timed like time_layer; None when the fused kernel does not take the shape."""
    dev = torch.device("cuda", torch.cuda.current_device())
    y2_elems = L.N * C2 * L.H_out * L.W_out
    per = 4 * (L.x_elems + y2_elems)
    nbuf = max(2, -(-min_cycle_bytes // per))
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        if not gconv.gconv_block_supported(d, C2):
            return None
        x0, w0 = synth.make_layer_tensors(min(L.N, 2), L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups, 99, L.x_dist)
        _, w2 = synth.make_layer_tensors(1, L.C_out, 1, 1, C2, 1, 1, 1, 98)
        reps_x = -(-L.N // x0.shape[0])
        xs = [torch.from_numpy(x0).to(dev).repeat(reps_x, 1, 1, 1)[:L.N].contiguous() for _ in range(nbuf)]
        ys = [torch.empty(y2_elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
        wp = torch.empty(gconv.gconv_block_packed_bytes(d, C2) // 4, dtype=torch.float32, device=dev)
        with torch.cuda.stream(stream):
            gconv.gconv_block_pack_weights(d, C2, torch.from_numpy(w0).to(dev), torch.from_numpy(w2.reshape(C2, L.C_out)).to(dev), wp, stream)
            for i in range(min(nbuf, 5) + 3):
                gconv.gconv_block_forward(d, C2, xs[i % nbuf], wp, ys[i % nbuf], stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            graph = torch.cuda.CUDAGraph()
            stream.synchronize()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(reps):
                    gconv.gconv_block_forward(d, C2, xs[i % nbuf], wp, ys[i % nbuf], stream)
            graph.replay()
            stream.synchronize()
            times = []
            for _ in range(5):
                e0.record(stream)
                graph.replay()
                e1.record(stream)
                stream.synchronize()
                times.append(e0.elapsed_time(e1) / reps)
        st = gconv.gconv_last_status(d, stream)
        assert st == 0, gconv.status_string(st)
        return statistics.median(times)
    finally:
        gconv.gconv_desc_destroy(d)


def block_row(L, C2, ms_block, ms_grouped, ms_pointwise, peaks):
    """Fused grouped + pointwise block: its time against the HBM floor of the block (x in, y2 out), against the
    unfused pair as measured (the grouped layer and the pointwise layer, each timed alone through gconv_forward) and
    against that pair's floor (the grouped layer as measured, plus reading y1 and writing y2 at the HBM peak)."""
    hbm = peaks["hbm_gbs"] * 1e9
    pix = L.N * L.H_out * L.W_out
    bytes_block = 4 * (L.x_elems + pix * C2)
    flops = L.flops + 2 * pix * L.C_out * C2
    t_tensor = flops / (0.5 * peaks["bf16_tflops"] * 1e12)
    t_roof = max(bytes_block / hbm, t_tensor)
    unfused_floor_ms = ms_grouped + 4e3 * pix * (L.C_out + C2) / hbm
    return {"layer": L.name, "groups": L.groups, "N": L.N, "C2": C2, "ms": ms_block, "grouped_only_ms": ms_grouped,
            "pointwise_only_ms": ms_pointwise, "unfused_measured_ms": ms_grouped + ms_pointwise,
            "unfused_floor_ms": unfused_floor_ms, "gflops": flops / (ms_block * 1e-3) / 1e9,
            "gbs": bytes_block / (ms_block * 1e-3) / 1e9, "roofline_ms": t_roof * 1e3,
            "bound": "hbm" if bytes_block / hbm >= t_tensor else "tensor", "roofline_frac": t_roof / (ms_block * 1e-3)}


def chained_stack_ms(torch, gconv, groups, stream, reps=50, family="wrn"):
    """Batch-1 inference over a stack as a real chain (each layer reads the previous layer's output), replayed as one
    CUDA graph: ms per pass.  This is the shape of the paper's whole-network timings (N = 1, Tables I and II),
    restricted to the grouped 3x3 layers: the 18-layer WRN-40-2-shaped stack, or the seven ResNet-34-shaped layers in
    network order (56x56 down to 7x7 through the stride-2 transitions)."""
    dev = torch.device("cuda", torch.cuda.current_device())
    layers = []
    for L in (wl.wrn_stack(groups, 1) if family == "wrn" else wl.resnet34_layers(groups, 1)):
        layers.extend([L] * L.repeat)
    descs, wps, bufs, wss = [], [], [], []
    x0, _ = synth.make_layer_tensors(1, layers[0].C_in, layers[0].H, layers[0].W, layers[0].C_out, 3, 3, groups, 3)
    bufs.append(torch.from_numpy(x0).to(dev).reshape(-1))
    try:
        for i, L in enumerate(layers):
            d = gconv.gconv_desc_create(*L.desc_args())
            descs.append(d)
            wss.append(attach_workspace(d, dev))
            _, w = synth.make_layer_tensors(1, L.C_in, L.H, L.W, L.C_out, 3, 3, groups, 100 + i)
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp, stream)
            wps.append(wp)
            bufs.append(torch.empty(L.y_elems, dtype=torch.float32, device=dev))

        def run():
            for i, d in enumerate(descs):
                gconv.gconv_forward(d, bufs[i], wps[i], bufs[i + 1], stream)

        with torch.cuda.stream(stream):
            for _ in range(3):
                run()
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                run()
            graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            e0.record(stream)
            for _ in range(reps):
                graph.replay()
            e1.record(stream)
            stream.synchronize()
        for d in descs:
            assert gconv.gconv_last_status(d, stream) == 0
        return e0.elapsed_time(e1) / reps
    finally:
        for d in descs:
            gconv.gconv_desc_destroy(d)


def graph_time_ms(torch, stream, body, reps, rounds=5):
    """Median device time (ms) of one call of `body(i)` when `reps` calls are replayed as one CUDA graph."""
    with torch.cuda.stream(stream):
        for i in range(3):
            body(i)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(reps):
                body(i)
        graph.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        times = []
        for _ in range(rounds):
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            times.append(e0.elapsed_time(e1) / reps)
    return statistics.median(times)


def launch_interval_us(torch, stream):
    """Latency floor: the interval between dependent launches of a kernel that does nothing to speak of (torch adds 1
    to a one-element tensor), 200 of them in one CUDA graph.  Off the product path."""
    t = torch.zeros(1, dtype=torch.float32, device=torch.device("cuda", torch.cuda.current_device()))
    return 1e3 * graph_time_ms(torch, stream, lambda i: t.add_(1.0), reps=200)


class CopyFloor:
    """Plain-copy floor of a layer: a torch copy kernel that moves the layer's algorithmic bytes (half read, half
    written), launched like the layer (one CUDA graph of back-to-back launches over rotating cold buffers)."""

    def __init__(self, torch, stream):
        self.torch, self.stream, self.cache = torch, stream, {}

    def ms(self, nbytes, reps=20):
        torch = self.torch
        elems = max(1, int(nbytes) // 8)          # elems read + elems written = nbytes
        if elems not in self.cache:
            dev = torch.device("cuda", torch.cuda.current_device())
            nbuf = max(2, -(-(2 * L2_BYTES + (64 << 20)) // (8 * elems)))
            src = [torch.empty(elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
            dst = [torch.empty(elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
            self.cache[elems] = graph_time_ms(torch, self.stream, lambda i: dst[i % nbuf].copy_(src[i % nbuf]), reps=max(reps, nbuf))
            del src, dst
        return self.cache[elems]


def tf32_probe_tflops(torch):
    """Measured TF32 tensor throughput of the box: one cuBLAS fp32 matmul of 8192^3 with TF32 enabled, best of 10
    (a context figure beside the roofline denominator, which stays half of the measured bf16 peak).  Off the product path."""
    dev = torch.device("cuda", torch.cuda.current_device())
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        n = 8192
        a = torch.randn(n, n, device=dev)
        b = torch.randn(n, n, device=dev)
        c = torch.empty(n, n, device=dev)
        for _ in range(3):
            torch.matmul(a, b, out=c)
        best = 1e9
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(10):
            e0.record()
            torch.matmul(a, b, out=c)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old


def targets_of(rows, monotone):
    """The three acceptance properties over every per-layer row: wide (tensor-bound) layers at >= 50 % of the TF32
    roofline, narrow-group and depthwise (HBM-bound) layers at >= 60 % of the HBM roofline, and time non-increasing in
    the group count.  Rows whose roofline time is below the launch-interval floor are listed but flagged."""
    def fails(bound, bar):
        out = []
        for r in rows:
            if r["bound"] == bound and r["roofline_frac"] < bar:
                out.append({"layer": r["layer"], "groups": r["groups"], "N": r["N"], "frac": round(r["roofline_frac"], 3),
                            "latency_bound": r.get("latency_bound", False)})
        return out
    wide, narrow = fails("tensor", 0.5), fails("hbm", 0.6)
    n_wide = sum(1 for r in rows if r["bound"] == "tensor")
    n_narrow = sum(1 for r in rows if r["bound"] == "hbm")
    return {"wide_ge_50pct_tf32": {"met": not wide, "rows": n_wide, "failing": wide},
            "narrow_ge_60pct_hbm": {"met": not narrow, "rows": n_narrow, "failing": narrow},
            "monotone": {"met": all(monotone.values()), "failing": sorted(k for k, v in monotone.items() if not v)}}


def layer_row(L, ms, variant, peaks, gconv):
    """Per-layer line of the metric: ms, GFLOP/s, achieved GB/s on compulsory bytes, % of roofline."""
    tf32_peak = 0.5 * peaks["bf16_tflops"] * 1e12
    fp32_peak = 148 * 128 * 2 * 1.965e9
    pipe_peak = tf32_peak if variant == gconv.GCONV_VARIANT_IGEMM_TF32 else fp32_peak
    t_hbm = L.compulsory_bytes / (peaks["hbm_gbs"] * 1e9)
    t_pipe = L.flops / pipe_peak
    t_roof = max(t_hbm, t_pipe)
    return {"layer": L.name, "groups": L.groups, "N": L.N, "Cg": L.Cg, "Kg": L.Kg, "variant": gconv.variant_name(variant),
            "ms": ms, "gflops": L.flops / (ms * 1e-3) / 1e9, "gbs": L.compulsory_bytes / (ms * 1e-3) / 1e9,
            "roofline_ms": t_roof * 1e3, "bound": "hbm" if t_hbm >= t_pipe else ("tensor" if pipe_peak == tf32_peak else "alu"),
            "roofline_frac": t_roof / (ms * 1e-3)}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2006_09791_b200 import build as gbuild
    from paper_2006_09791_b200 import gconv

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libgconv has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        gbuild.build()
    if world > 1:
        dist.barrier()
    gconv.load()
    peaks = load_peaks()
    stream = torch.cuda.Stream(device=dev)

    # ---- set up the step: every layer instance with its own buffers --------------------------------
    plan = step_layers(BATCH)
    host_x, host_y, dev_w = {}, {}, {}
    insts = []
    for g, L in plan:
        key = (L.name, g)
        if key not in host_x:
            x2, w = synth.make_layer_tensors(2, L.C_in, L.H, L.W, L.C_out, 3, 3, g, synth.layer_seed(2, L.C_in, L.H, L.C_out, g))
            hx = torch.from_numpy(x2).repeat(BATCH // 2, 1, 1, 1).contiguous().pin_memory()
            host_x[key] = hx
            host_y[key] = torch.empty(L.y_elems, dtype=torch.float32).pin_memory()
            d = gconv.gconv_desc_create(*L.desc_args())
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
            gconv.gconv_desc_destroy(d)
            dev_w[key] = wp
        insts.append(Instance(g, L, host_x[key].to(dev), dev_w[key], torch, gconv))
    torch.cuda.synchronize()
    step_macs = sum(i.L.macs for i in insts)
    step_flops = 2 * step_macs
    launches_per_step = sum(gconv.gconv_forward_launches(i.desc) for i in insts)

    def step_device():
        for it in insts:
            gconv.gconv_forward(it.desc, it.x, it.wp, it.y, stream)

    # The host-buffer path is issued round-robin on three streams so that one layer's upload, another's kernel and a
    # third's download overlap (PCIe is full duplex); layers that share a host output buffer share a stream.
    e2e_streams = [stream, torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]
    key_stream = {}
    for it in insts:
        key_stream.setdefault((it.L.name, it.g), e2e_streams[len(key_stream) % len(e2e_streams)])

    def step_host():
        for it in insts:
            key = (it.L.name, it.g)
            gconv.gconv_forward_host(it.desc, host_x[key], it.wp, host_y[key], it.x, it.y, key_stream[key])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        return reduce_max_over_ranks(ms, world, dev)

    # ---- device-resident timing: the step as one CUDA graph ----------------------------------------
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step_device()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step_device()
        graph.replay()
        stream.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        e1.record(stream)
    barrier()
    ms_dev = max_over_ranks(e0.elapsed_time(e1) / args.steps)
    clocks = sampler.stop()
    for it in insts:
        st = gconv.gconv_last_status(it.desc, stream)
        assert st == 0, gconv.status_string(st)

    # ---- the same step with the five stacks (independent networks) spread over two streams ----------------
    # Reported beside the headline, not as it: layers of a stack stay in stream order, stacks of different group counts
    # share no data, so a second stream lets one stack's kernels fill the gaps between the other's dependent launches.
    side = torch.cuda.Stream(device=dev)

    def step_two_streams():
        fork = torch.cuda.Event()
        fork.record(stream)
        side.wait_event(fork)
        for k, g in enumerate(wl.WRN_GROUPS):
            s_k = stream if k % 2 == 0 else side
            for it in insts:
                if it.g == g:
                    gconv.gconv_forward(it.desc, it.x, it.wp, it.y, s_k)
        join = torch.cuda.Event()
        join.record(side)
        stream.wait_event(join)

    with torch.cuda.stream(stream):
        for _ in range(3):
            step_two_streams()
        stream.synchronize()
        side.synchronize()
        graph2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph2, stream=stream):
            step_two_streams()
        graph2.replay()
        stream.synchronize()
    barrier()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            graph2.replay()
        e1.record(stream)
    barrier()
    ms_two = max_over_ranks(e0.elapsed_time(e1) / args.steps)
    for it in insts:
        st = gconv.gconv_last_status(it.desc, stream)
        assert st == 0, gconv.status_string(st)

    # ---- end to end through the host-buffer entry point --------------------------------------------
    for _ in range(2):
        step_host()
    e2e_steps = max(1, min(args.steps, 10))
    barrier()
    e0.record(stream)
    for st_ in e2e_streams[1:]:
        st_.wait_event(e0)
    for _ in range(e2e_steps):
        step_host()
    for st_ in e2e_streams[1:]:
        done = torch.cuda.Event()
        done.record(st_)
        stream.wait_event(done)
    e1.record(stream)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1) / e2e_steps)
    h2d = sum(4 * i.L.x_elems for i in insts)
    d2h = sum(4 * i.L.y_elems for i in insts)

    # ---- per-layer table (the metric proper) and roofline of the dominant kernel --------------------
    rows, extra = [], {}
    if rank == 0 and not args.no_layers:
        floor_us = launch_interval_us(torch, stream)
        copy_floor = CopyFloor(torch, stream)

        def measured_row(L, reps):
            """One per-layer row: cold-L2 time (the one the roofline fraction uses), warm-L2 time, the plain-copy floor
            for the same bytes and the launch-interval floor; `latency_bound` marks rows whose roofline time is below
            the launch interval."""
            ms, v = time_layer(torch, gconv, L, stream, reps=reps)
            row = layer_row(L, ms, v, peaks, gconv)
            if not args.quick:
                row["ms_warm"] = time_layer(torch, gconv, L, stream, reps=20, warm=True)[0]
                row["copy_floor_ms"] = copy_floor.ms(L.compulsory_bytes)
            row["launch_floor_ms"] = floor_us * 1e-3
            row["latency_bound"] = row["roofline_ms"] < floor_us * 1e-3
            return row, ms, v

        seen = {}
        for g, L in plan:
            key = (L.name, g)
            if key in seen:
                continue
            row, ms, v = measured_row(L, 160)
            seen[key] = (ms, v, L)
            rows.append(row)
        by_variant = {}
        for (name, g), (ms, v, L) in seen.items():
            a = by_variant.setdefault(v, {"ms": 0.0, "bytes": 0, "flops": 0, "launches": 0})
            a["ms"] += ms * L.repeat
            a["bytes"] += L.compulsory_bytes * L.repeat
            a["flops"] += L.flops * L.repeat
            a["launches"] += L.repeat
        dom_v = max(by_variant, key=lambda k: by_variant[k]["ms"])
        dom = by_variant[dom_v]
        t_hbm = dom["bytes"] / (peaks["hbm_gbs"] * 1e9)
        pipe_peak = 0.5 * peaks["bf16_tflops"] * 1e12 if dom_v == gconv.GCONV_VARIANT_IGEMM_TF32 else 148 * 128 * 2 * 1.965e9
        t_pipe = dom["flops"] / pipe_peak
        if t_hbm >= t_pipe:
            ach = dom["bytes"] / (dom["ms"] * 1e-3) / 1e9
            roofline = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"], "traffic": None}
        else:
            ach = dom["flops"] / (dom["ms"] * 1e-3) / 1e12
            roofline = {"bound": "tensor" if dom_v == gconv.GCONV_VARIANT_IGEMM_TF32 else "alu", "achieved": ach,
                        "peak": pipe_peak / 1e12, "unit": "TFLOP/s", "frac": ach / (pipe_peak / 1e12), "traffic": None}
        traffic = ncu_traffic().get(gconv.variant_name(dom_v))
        roofline["traffic"] = traffic["bytes"] if traffic else None
        roofline.update({"kernel": gconv.variant_name(dom_v), "launches_per_step": dom["launches"],
                         "algorithmic_bytes_per_launch": dom["bytes"] / dom["launches"],
                         "avg_launch_us": 1e3 * dom["ms"] / dom["launches"],
                         "share_of_step": dom["ms"] / sum(a["ms"] for a in by_variant.values()),
                         "peak_source": peaks["source"],
                         "traffic_source": ("ncu capture at commit %s (profiles/dram_traffic_per_launch.md)" % traffic["commit"]) if traffic else None})
        extra["roofline"] = roofline
        extra["floors"] = {"launch_interval_us": floor_us,
                           "step_copy_floor_ms": None if args.quick else sum(r["copy_floor_ms"] * seen[(r["layer"], r["groups"])][2].repeat for r in rows),
                           "how": "launch interval: a one-element torch kernel, 200 dependent launches in one CUDA graph; copy floor: a torch "
                                  "copy kernel moving each layer's algorithmic bytes, launched like the layer (graph, cold rotating buffers)"}
        # time per group count (the paper's acceptance property: time falls as g rises)
        extra["ms_by_groups"] = {str(g): sum(ms * L.repeat for (n, gg), (ms, v, L) in seen.items() if gg == g)
                                 for g in wl.WRN_GROUPS}
        monotone = {}
        by_shape = {}
        for (name, g), (ms, v, L) in seen.items():
            by_shape.setdefault(name, []).append((g, ms))
        for name, t in by_shape.items():
            t = [ms for g, ms in sorted(t)]
            monotone["wrn:" + name] = all(b <= 1.03 * a for a, b in zip(t, t[1:]))
        graded = list(rows)
        if world == 1 and not args.quick:
            # ---- the other benchmark families, at the batch the problem statement names for them ----------------
            (L0,) = wl.config0()
            extra["config0_layer"] = [measured_row(L0, 160)[0]]
            sweep_rows = [measured_row(L, 20)[0] for L in wl.sweep_layers(32)]
            extra["sweep_layers"] = sweep_rows
            t = [r["ms"] for r in sweep_rows]
            monotone["sweep_256@56"] = all(b <= 1.03 * a for a, b in zip(t, t[1:]))
            extra["resnext_layers"] = [measured_row(L, 20)[0] for L in wl.resnext_layers(64)]
            # ResNet-34-shaped layers at N = 64 for every group count, with the time-falls-with-groups check per shape
            r34_rows, r34_ms = [], {}
            for g in wl.R34_GROUPS:
                for L in wl.resnet34_layers(g, 64):
                    row, ms, v = measured_row(L, 20)
                    r34_rows.append(row)
                    r34_ms.setdefault(L.name, []).append(ms)
            extra["resnet34_layers"] = r34_rows
            extra["resnet34_monotone"] = {name: all(b <= 1.03 * a for a, b in zip(t, t[1:])) for name, t in r34_ms.items()}
            for name, ok in extra["resnet34_monotone"].items():
                monotone["r34:" + name] = ok
            graded += extra["config0_layer"] + sweep_rows + extra["resnext_layers"] + r34_rows
            extra["depthwise_and_pointwise_layers"] = [measured_row(L, 20)[0] for L in wl.mobilenetv2_dw_layers(64) + wl.depthwise5x5_layers(64) + wl.pointwise_layers(64)]
            block_rows = []
            for L, C2 in wl.fused_blocks():
                msb = time_block(torch, gconv, L, C2, stream)
                if msb is not None:
                    msg, _ = time_layer(torch, gconv, L, stream, reps=20)
                    Lp = wl.Layer(L.name + "_pw", L.N, L.C_out, L.H_out, L.W_out, C2, 1, 1, 1, 0, 1, 1)
                    msp, _ = time_layer(torch, gconv, Lp, stream, reps=20)
                    block_rows.append(block_row(L, C2, msb, msg, msp, peaks))
            extra["fused_blocks"] = block_rows
            # batch-1 whole-stack timings as real chains in one CUDA graph (the shape of the paper's Tables I and II)
            extra["stack_n1_chained_ms_by_groups"] = {str(g): chained_stack_ms(torch, gconv, g, stream) for g in wl.WRN_GROUPS}
            extra["resnet34_n1_chained_ms_by_groups"] = {str(g): chained_stack_ms(torch, gconv, g, stream, family="r34") for g in wl.R34_GROUPS}
            extra["peaks"] = {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"], "tf32_tflops_used": 0.5 * peaks["bf16_tflops"],
                              "tf32_tflops_cublas_probe": tf32_probe_tflops(torch), "tf32_tflops_nominal": 1100.0,
                              "fp32_ffma_tflops": 148 * 128 * 2 * 1.965e9 / 1e12, "source": peaks["source"]}
        extra["targets"] = targets_of(graded, monotone)

    # ---- CPU baselines (rank 0, N=1 only) ----------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        threads = min(oracle.max_threads(), len(os.sched_getaffinity(0)))
        secs, macs = oracle_sample_time(CPU_LEG_BATCH, threads)
        cpu = {"value": 2.0 * macs / secs / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": secs,
               "sample": "the 18-layer stack at N=%d (of %d) for every group count, oracle as it stands" % (CPU_LEG_BATCH, BATCH)}
        s1, m1 = oracle_sample_time(1, 1)
        cpu["single_thread"] = {"value": 2.0 * m1 / s1 / 1e9, "unit": UNIT, "cores": 1, "seconds": s1,
                                "sample": "the same stack at N=1, one thread"}
        extra["cpu_baseline_gspc"] = gspc_baseline(threads)

    if rank == 0:
        line = {"metric": METRIC, "value": aggregate_value(step_flops, world, ms_dev), "unit": UNIT, "n_gpus": world,
                "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_dev, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32+tf32", "data": "synthetic",
                "config": {"workload": WORKLOAD, "layers_per_step": len(insts), "batch": BATCH, "groups": list(wl.WRN_GROUPS),
                           "parallelism": "replicas only (%d)" % world, "launch": "cuda graph of the step",
                           "l2": "every layer instance owns its x/y buffers: %.2f GB cycled per step > 126 MB L2"
                                 % ((h2d + d2h) / 1e9)},
                "clocks": clocks,
                "e2e": {"value": aggregate_value(step_flops, world, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
                        "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
                "two_streams": {"ms_per_step": ms_two, "value": aggregate_value(step_flops, world, ms_two), "unit": UNIT,
                                "how": "the same 90 launches in one CUDA graph, group counts 1, 4, 16 on one stream and 2, 8 on a second"},
                "gpu_launches": launches_per_step * args.steps,
                "cpu_baseline": cpu, "layers": rows}
        line.update(extra)
        print(json.dumps(line))
    for it in insts:
        gconv.gconv_desc_destroy(it.desc)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="accepted for compatibility: the sweep tables are part of the default run")
    ap.add_argument("--quick", action="store_true", help="only the step and its own layer table (no other families, no warm/copy columns)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-layers", action="store_true", help="skip the per-layer table (short runs under a profiler)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
