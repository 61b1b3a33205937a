#!/usr/bin/env python
"""Benchmark of the dynamic-weight-slicing hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: gate (average pool,
FC-ReLU-FC, arg-max) -> routing (stable grouping) -> the block's sliced grouped GEMMs -> outputs in
input order.  Default workload: ResNet-50 stage-3 dynamic bottleneck, bf16 NHWC, batch 128, 14x14,
1x1 1024->w, 3x3 w->w, 1x1 w->1024 with 14 inner widths, gate-driven routing.

Prints ONE JSON line (see --help).  `value` is executed TFLOP/s of the whole step (2 x multiply-adds
of the sliced layers actually run, divided by the step time, gate and routing included), inputs
resident in HBM.  `e2e` is the same metric with the batch starting and ending in pinned host memory.
`roofline` describes the grouped-GEMM kernel, `cpu_baseline` the fp64 CPU oracle on a bounded sample.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0
CHAIN_CFG2_DRAM_BYTES = 68.5e6   # per launch of gemm_bf16_chain_kernel on cfg2, B = 128 (57.6 MB read + 10.9 MB written)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# --------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.samples.append(line.strip())
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.samples:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------- workloads
class Bottleneck:
    """ResNet-50-style dynamic bottleneck (configs 2 and 4)."""

    def __init__(self, dsn, torch, dev, cfg, gate_driven=True, copies=None):
        import dsn_workloads as wl
        self.dsn, self.torch, self.dev, self.cfg = dsn, torch, dev, cfg
        B, H, Wd, C, Ci, T = cfg["B"], cfg["H"], cfg["W"], cfg["C_outer"], cfg["C_inner"], cfg["T"]
        self.B, self.R, self.C, self.T, self.widths = B, H * Wd, C, T, cfg["widths"]
        self.gate_driven = gate_driven
        up = lambda a: torch.from_numpy(wl.bf16_bits(np.ascontiguousarray(a)).view(np.int16)).to(dev).view(torch.bfloat16)
        self.x_host_bits = wl.bf16_bits(cfg["x"]).view(np.int16)
        x_bytes = self.x_host_bits.nbytes
        self.copies = copies or max(2, -(-2 * L2_BYTES // (2 * x_bytes)) + 1)   # inputs + outputs rotate past L2
        self.xs = [torch.from_numpy(self.x_host_bits).to(dev).view(torch.bfloat16).reshape(B, H, Wd, C)
                   for _ in range(self.copies)]
        self.ys = [torch.zeros(B, H, Wd, C, dtype=torch.bfloat16, device=dev) for _ in range(self.copies)]
        self.W1 = up(cfg["W1"].reshape(Ci, C))
        self.W2 = up(np.transpose(cfg["W2"], (0, 2, 3, 1)))
        self.W3 = up(cfg["W3"].reshape(C, Ci))
        full = [C] * T
        self.slices = [(full, self.widths, 1), (self.widths, self.widths, 3), (self.widths, full, 1)]
        mk = dsn.make_conv_desc
        self.layers = [mk(dsn.BF16, H, Wd, 1, 0, C, Ci, full, self.widths, self.W1, act=dsn.ACT_RELU),
                       mk(dsn.BF16, H, Wd, 3, 1, Ci, Ci, self.widths, self.widths, self.W2, act=dsn.ACT_RELU),
                       mk(dsn.BF16, H, Wd, 1, 0, Ci, C, self.widths, full, self.W3)]
        self.gW1 = torch.from_numpy(cfg["gate_W1"]).to(dev)
        self.gW2 = torch.from_numpy(cfg["gate_W2"]).to(dev)
        self.gate = dsn.make_gate_desc(dsn.BF16, B, self.R, C, self.gW1.shape[0], T, self.gW1, self.gW2)
        self.idx_given = torch.from_numpy(cfg["idx"]).to(dev)
        self.L = dsn.make_layer_desc(B, T, self.layers, self.gate if gate_driven else None)
        self.ws = torch.empty(dsn.dsn_layer_workspace_bytes(self.L), dtype=torch.uint8, device=dev)
        self.idx_out = torch.zeros(B, dtype=torch.int32, device=dev)
        # decomposed form (same kernels, one C call per step of the path) for per-kernel timing
        self.gate_ws = torch.empty(dsn.dsn_gate_workspace_bytes(self.gate), dtype=torch.uint8, device=dev)
        ints = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
        self.routing = dsn.make_routing(B, T, ints(T), ints(T + 1), ints(B), ints(B))
        self.t1 = torch.zeros(B, H, Wd, Ci, dtype=torch.bfloat16, device=dev)
        self.t2 = torch.zeros(B, H, Wd, Ci, dtype=torch.bfloat16, device=dev)
        self.dec_layers = [
            mk(dsn.BF16, H, Wd, 1, 0, C, Ci, full, self.widths, self.W1, act=dsn.ACT_RELU, in_order=0, out_order=1),
            mk(dsn.BF16, H, Wd, 3, 1, Ci, Ci, self.widths, self.widths, self.W2, act=dsn.ACT_RELU, in_order=1, out_order=1),
            mk(dsn.BF16, H, Wd, 1, 0, Ci, C, self.widths, full, self.W3, in_order=1, out_order=0)]
        # small batches run the three layers as one chained launch (every CTA pair owns whole samples)
        self.chained = os.environ.get("DSN_CHAIN", "1") != "0" and B <= 148 and 150 <= self.R <= 256
        self.L_given = dsn.make_layer_desc(B, T, self.layers, None)
        # launches per step: gate = pool + hidden + score, route, then one chained launch or three GEMMs
        self.kernels_per_step = (3 if gate_driven else 0) + 1 + (1 if self.chained else 3)
        self.name = cfg["name"]

    def step(self, ctx, i):
        k = i % self.copies
        self.dsn.dsn_layer_forward(ctx, self.L, self.xs[k], None if self.gate_driven else self.idx_given, self.ys[k],
                                   self.ws, idx_out=self.idx_out)

    def _parts(self):
        d = self.dsn
        parts = []
        if self.gate_driven:
            parts.append(("gate", lambda ctx, k: d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws)))
            parts.append(("route", lambda ctx, k: d.dsn_route(ctx, self.idx_out, self.B, self.T, self.routing)))
        else:
            parts.append(("route", lambda ctx, k: d.dsn_route(ctx, self.idx_given, self.B, self.T, self.routing)))
        if self.chained:
            # the step's own GEMM launch cannot be called without its routing: timed together with the route
            # kernel (dsn_layer_forward on given indices); the three single-layer calls below are reference points
            src = self.idx_out if self.gate_driven else self.idx_given
            parts.append(("route+gemm_chain", lambda ctx, k: d.dsn_layer_forward(ctx, self.L_given, self.xs[k], src, self.ys[k], self.ws)))
        parts.append(("gemm:conv1_1x1", lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[0], self.routing, self.xs[k], self.t1)))
        parts.append(("gemm:conv2_3x3", lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[1], self.routing, self.t1, self.t2)))
        parts.append(("gemm:conv3_1x1", lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[2], self.routing, self.t2, self.ys[k])))
        return parts

    def decomposed_step(self, ctx, i, mark):
        """Same path as separate C calls; mark(name) is called after each."""
        k = i % self.copies
        mark("start")
        for name, fn in self._parts():
            fn(ctx, k)
            mark(name)

    def decomposed_part(self, ctx, i, part):
        self._parts()[part][1](ctx, i % self.copies)

    def histogram(self):
        return np.bincount(self.idx_out.cpu().numpy() if self.gate_driven else self.cfg["idx"], minlength=self.T)

    def exec_flops(self, counts):
        return sum(2 * self.dsn.dsn_executed_macs(counts.tolist(), self.R, ki, ko, K) for ki, ko, K in self.slices)

    def gemm_bytes(self, counts):
        """Algorithmic bytes of the three GEMM launches: sliced input read once, sliced output written
        once, each used weight slice read once (bf16)."""
        total = 0
        for ki, ko, K in self.slices:
            for t, n in enumerate(counts):
                if n:
                    total += 2 * (int(n) * self.R * (ki[t] + ko[t]) + ki[t] * ko[t] * K * K)
        return total

    def e2e_io(self):
        t = self.torch
        hx = t.from_numpy(self.x_host_bits.copy()).pin_memory()
        hy = t.empty(self.ys[0].numel(), dtype=t.int16).pin_memory()
        return hx, hy

    def e2e_step(self, ctx, hx, hy):
        t = self.torch
        self.xs[0].view(t.int16).view(-1).copy_(hx.view(-1), non_blocking=True)
        self.step(ctx, 0)
        hy.copy_(self.ys[0].view(t.int16).view(-1), non_blocking=True)

    def e2e_pipeline(self, ctx, hx, hy, n, streams, events):
        """n steps with the batch starting and ending in pinned host memory: the upload of step i+1, the
        compute of step i and the download of step i-1 run on three streams over the rotating buffer sets."""
        t = self.torch
        s_up, s_run, s_down = streams
        for i in range(n):
            k = i % self.copies
            up_done, run_done, down_done = events[k]
            with t.cuda.stream(s_up):
                s_up.wait_event(down_done)          # buffer set k is free again
                self.xs[k].view(t.int16).view(-1).copy_(hx.view(-1), non_blocking=True)
                up_done.record(s_up)
            with t.cuda.stream(s_run):
                s_run.wait_event(up_done)
                self.step(ctx, k)
                run_done.record(s_run)
            with t.cuda.stream(s_down):
                s_down.wait_event(run_done)
                hy.copy_(self.ys[k].view(t.int16).view(-1), non_blocking=True)
                down_done.record(s_down)

    def oracle_sample(self, n):
        """Times the fp64 oracle on the first n samples (gate + bottleneck chain)."""
        from oracle import dsn_oracle as O
        cfg = self.cfg
        x = cfg["x"][:n]
        t0 = time.perf_counter()
        idx, _, _ = O.gate(x.reshape(n, self.R, self.C), cfg["gate_W1"], cfg["gate_W2"])
        if not self.gate_driven:
            idx = cfg["idx"][:n]
        O.route(idx, self.T)
        O.bottleneck(x, cfg["W1"], cfg["W2"], cfg["W3"], idx, self.widths, mirror_bf16=True)
        dt = time.perf_counter() - t0
        flops = sum(2 * O.executed_macs(idx, self.R, ki, ko, K) for ki, ko, K in self.slices)
        return flops, dt


def make_workload(name, dsn, torch, dev, batch=None):
    import dsn_workloads as wl
    if name == "cfg2":
        return Bottleneck(dsn, torch, dev, wl.config2(B=batch or 128), gate_driven=True)
    if name.startswith("cfg4-stage"):
        stage = int(name[len("cfg4-stage")])
        routing = "uniform" if name.endswith("uniform") else "skewed"
        return Bottleneck(dsn, torch, dev, wl.config4(stage, B=batch or 256, routing=routing), gate_driven=False)
    raise SystemExit(f"unknown workload {name}")


# --------------------------------------------------------------------------------------------- reference arm
def run_reference(args):
    """Times the CPU oracle (the only 'reference implementation' this method has) on host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import dsn_workloads as wl
    from oracle import dsn_oracle as O
    cfg = wl.config2(B=128)
    n = 8
    R, C, T, widths = cfg["H"] * cfg["W"], cfg["C_outer"], cfg["T"], cfg["widths"]
    full = [C] * T
    slices = [(full, widths, 1), (widths, widths, 3), (widths, full, 1)]

    def one(i):
        x = cfg["x"][(i * n) % 128:(i * n) % 128 + n]
        idx, _, _ = O.gate(x.reshape(n, R, C), cfg["gate_W1"], cfg["gate_W2"])
        O.route(idx, T)
        O.bottleneck(x, cfg["W1"], cfg["W2"], cfg["W3"], idx, widths, mirror_bf16=True)
        return sum(2 * O.executed_macs(idx, R, ki, ko, K) for ki, ko, K in slices)

    for i in range(args.warmup):
        one(i)
    flops, t0 = 0, time.perf_counter()
    for i in range(args.steps):
        flops += one(i)
    dt = time.perf_counter() - t0
    val = flops / dt / 1e12
    cores = os.cpu_count()
    print(json.dumps({
        "impl": "reference", "metric": "sliced_gemm_executed_tflops", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg2 ResNet-50 stage-3 dynamic bottleneck, bf16-valued inputs, 14x14, 14 widths",
                   "sample": f"{n} samples per step"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": f"{n} of 128 samples per step, {args.steps} steps"},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))



# --------------------------------------------------------------------------------------------- per-layer table
def run_table(args):
    """Per-layer numbers for every configuration (markdown table rows): CUDA-graph replay over
    rotating buffers larger than L2, executed TFLOP/s, fraction of the shape's roofline bound."""
    import torch
    from paper_2109_10060_b200.build import build
    build()
    import paper_2109_10060_b200 as dsn
    import dsn_workloads as wl
    from oracle import dsn_oracle as O
    dev = torch.device("cuda:0")
    ctx = dsn.Context(0)
    peaks = load_peaks()
    PEAK, HBM = peaks["bf16_tflops"], peaks["hbm_gbs"]
    ints = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    side = torch.cuda.Stream()

    def graph_time(call, nbuf, reps=10):
        with torch.cuda.stream(side):
            call(0)
        torch.cuda.synchronize()
        if args.no_graph:   # direct calls (for profilers): two passes over the buffers, the second one timed
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(side):
                for i in range(nbuf):
                    call(i)
                e0.record(side)
                for i in range(nbuf):
                    call(i)
                e1.record(side)
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / nbuf * 1e3
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for i in range(nbuf):
                call(i)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * nbuf) * 1e3  # us

    print("| config | layer | routing | us | executed TFLOP/s | % measured BF16 peak | bound (TFLOP/s) | % of bound | GB/s | samples/s |")
    print("|---|---|---|---|---|---|---|---|---|---|")

    import re
    want = (lambda *names: re.search(args.table_filter, " ".join(names)) is not None) if args.table_filter else (lambda *names: True)
    div = max(1, args.table_batch_div)

    def layer(cfgname, lname, rname, B, H, Cin, Cout, k_in, k_out, idx, K=1, act=0, orders=(1, 1), group_list=None):
        if not want(cfgname, lname, rname):
            return
        if div > 1:
            if group_list is not None:
                return
            B = B // div
            idx = idx[:B]
        T = len(k_in)
        R = H * H if K == 3 else H
        if group_list is None:
            r = dsn.make_routing(B, T, ints(np.zeros(T)), ints(np.zeros(T + 1)), ints(np.zeros(B)), ints(np.zeros(B)))
            dsn.dsn_route(ctx, ints(idx), B, T, r)
        else:
            r = group_list
        per = B * R * (Cin + Cout) * 2
        nbuf = max(2, int(2.2 * L2_BYTES // per) + 1)
        xs = [torch.randn(B, R, Cin, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        ys = [torch.zeros(B, R, Cout, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        if K == 1:
            W = (torch.randn(Cout, Cin, device=dev) * Cin ** -0.5).to(torch.bfloat16)
            d = dsn.make_linear_desc(dsn.BF16, R, Cin, Cout, k_in, k_out, W, act=act, in_order=orders[0], out_order=orders[1])
            call = lambda i: dsn.dsn_sliced_linear(ctx, d, r, xs[i % nbuf], ys[i % nbuf])
        else:
            W = (torch.randn(Cout, K, K, Cin, device=dev) * (Cin * K * K) ** -0.5).to(torch.bfloat16)
            d = dsn.make_conv_desc(dsn.BF16, H, H, K, 1, Cin, Cout, k_in, k_out, W, act=act, in_order=orders[0],
                                   out_order=orders[1])
            call = lambda i: dsn.dsn_sliced_conv(ctx, d, r, xs[i % nbuf], ys[i % nbuf])
        us = graph_time(call, nbuf)
        code, _ = ctx.get_status()
        assert code == 0, code
        counts = np.bincount(idx, minlength=T)
        flops = 2 * dsn.dsn_executed_macs(counts.tolist(), R, k_in, k_out, K)
        byts = sum(2 * (int(n) * R * (k_in[t] + k_out[t]) + k_in[t] * k_out[t] * K * K) for t, n in enumerate(counts) if n)
        tf = flops / us / 1e6
        bound = min(PEAK, flops / byts * HBM / 1e3)
        print(f"| {cfgname} | {lname} | {rname} | {us:.1f} | {tf:.0f} | {100 * tf / PEAK:.1f} | {bound:.0f} | "
              f"{100 * tf / bound:.0f} | {byts / us / 1e3:.0f} | {B / us * 1e6:.0f} |", flush=True)
        del xs, ys

    def gate_route(cfgname, B, R, C, T):
        if not want(cfgname, "gate route", "-"):
            return
        B = B // div
        per = B * R * C * 2
        nbuf = max(2, int(2.2 * L2_BYTES // per) + 1)
        xs = [torch.randn(B, R, C, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        W1 = torch.randn(128, C, device=dev) * C ** -0.5
        W2 = torch.randn(T, 128, device=dev) * 128 ** -0.5
        g = dsn.make_gate_desc(dsn.BF16, B, R, C, 128, T, W1, W2)
        ws = torch.empty(dsn.dsn_gate_workspace_bytes(g), dtype=torch.uint8, device=dev)
        idx = torch.zeros(B, dtype=torch.int32, device=dev)
        r = dsn.make_routing(B, T, ints(np.zeros(T)), ints(np.zeros(T + 1)), ints(np.zeros(B)), ints(np.zeros(B)))
        us = graph_time(lambda i: dsn.dsn_gate(ctx, g, xs[i % nbuf], idx, None, ws), nbuf)
        print(f"| {cfgname} | gate (pool + FC-ReLU-FC + arg-max) | - | {us:.1f} | - | - | HBM {HBM:.0f} GB/s | "
              f"{100 * per / us / 1e3 / HBM:.0f} | {per / us / 1e3:.0f} | {B / us * 1e6:.0f} |", flush=True)
        us = graph_time(lambda i: dsn.dsn_route(ctx, idx, B, T, r), 8)
        print(f"| {cfgname} | route | - | {us:.1f} | - | - | launch latency | - | - | {B / us * 1e6:.0f} |", flush=True)

    # config 2 / 4: bottlenecks
    for cfgname, B, stages in (("cfg2", 128, (3,)), ("cfg4", 256, (1, 2, 3, 4))):
        for stage in stages:
            hw, outer, inner = wl.RESNET_STAGES[stage]
            widths = wl.WIDTHS_14[inner]
            full = [outer] * 14
            routings = [("uniform", wl.idx_quota_uniform(wl.rng(40 + stage, 6), B, 14))]
            if cfgname == "cfg4":
                routings.insert(0, ("skewed", wl.idx_skewed_bands(wl.rng(40 + stage, 6), B, 14)))
            tag = f"{cfgname} {hw}x{hw}"
            gate_route(tag, B, hw * hw, outer, 14)
            for rname, idx in routings:
                layer(tag, f"conv1 1x1 {outer}->w", rname, B, hw * hw, outer, inner, full, widths, idx, act=1)
                layer(tag, "conv2 3x3 w->w", rname, B, hw, inner, inner, widths, widths, idx, K=3, act=1)
                layer(tag, f"conv3 1x1 w->{outer}", rname, B, hw * hw, inner, outer, widths, full, idx)
    # config 3: ViT-S style
    B, paths = 256, wl.vit_small_paths()
    idx = wl.idx_quota_uniform(wl.rng(3, 9), B, 48)
    gate_route("cfg3", B, 197, 384, 48)
    for lname, Cin, Cout, act in (("qkv", 384, 1152, 0), ("proj", 384, 384, 0), ("fc1", 384, 1536, 2), ("fc2", 1536, 384, 0)):
        ki, ko = wl.vit_layer_slices(paths, 64, lname)
        layer("cfg3", lname, "uniform", B, 197, Cin, Cout, ki, ko, idx, act=act)
    def attention(cfgname, B, N, H, heads, idx, rname):
        if not want(cfgname, "attention core", rname):
            return
        B = B // div
        idx = idx[:B]
        T = len(heads)
        r = dsn.make_routing(B, T, ints(np.zeros(T)), ints(np.zeros(T + 1)), ints(np.zeros(B)), ints(np.zeros(B)))
        dsn.dsn_route(ctx, ints(idx), B, T, r)
        per = B * N * 4 * H * 64 * 2
        nbuf = max(2, int(2.2 * L2_BYTES // per) + 1)
        qs = [torch.randn(B, N, 3 * H * 64, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        os_ = [torch.zeros(B, N, H * 64, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        d = dsn.make_attention_desc(N, H, 64, heads, order=dsn.GROUPED)
        us = graph_time(lambda i: dsn.dsn_sliced_attention(ctx, d, r, qs[i % nbuf], os_[i % nbuf]), nbuf)
        assert ctx.get_status()[0] == 0
        hsum = sum(heads[t] for t in idx)
        flops = 4.0 * N * N * 64 * hsum
        byts = 2.0 * N * 4 * 64 * hsum
        tf = flops / us / 1e6
        bound = min(PEAK, flops / byts * HBM / 1e3)
        print(f"| {cfgname} | attention core (N={N}) | {rname} | {us:.1f} | {tf:.0f} | {100 * tf / PEAK:.1f} | {bound:.0f} | "
              f"{100 * tf / bound:.0f} | {byts / us / 1e3:.0f} | {B / us * 1e6:.0f} |", flush=True)

    attention("cfg3", 256, 197, 6, [p_[1] for p_ in wl.vit_small_paths()], wl.idx_quota_uniform(wl.rng(3, 9), 256, 48), "uniform")
    attention("cfg5", 1024, 197, 12, [p_[1] for p_ in wl.vit_base_paths()], wl.idx_quota_uniform(wl.rng(5, 9), 1024, 8), "uniform")
    # config 5: ViT-B width
    B, paths = 1024, wl.vit_base_paths()
    gate_route("cfg5", B, 197, 768, 8)
    cases = [("all on path 7", wl.idx_all_one(B, 7)), ("all on path 0", wl.idx_all_one(B, 0)),
             ("uniform", wl.idx_quota_uniform(wl.rng(5, 9), B, 8)), ("zipf(1.2)", wl.idx_zipf(wl.rng(5, 9), B, 8))]
    for rname, idx in cases:
        for lname, Cin, Cout, act in (("qkv", 768, 2304, 0), ("fc1", 768, 3072, 2), ("fc2", 3072, 768, 0)):
            ki, ko = wl.vit_layer_slices(paths, 64, lname)
            layer("cfg5", lname, rname, B, 197, Cin, Cout, ki, ko, idx, act=act)
    # singleton groups: 1024 caller-built groups of one sample each
    idx = (np.arange(B) % 8).astype(np.int32)
    order = np.arange(B, dtype=np.int32)
    gl = dsn.make_routing(B, B, ints(np.ones(B)), ints(np.arange(B + 1)), ints(order), ints(order), ints(idx))
    for lname, Cin, Cout, act in (("qkv", 768, 2304, 0), ("fc1", 768, 3072, 2), ("fc2", 3072, 768, 0)):
        ki, ko = wl.vit_layer_slices(paths, 64, lname)
        layer("cfg5", lname, "1024 singleton groups", B, 197, Cin, Cout, ki, ko, idx, act=act, group_list=gl)
    # MobileNet-shaped pointwise layers (supplement)
    for hw, C in ((14, 640), (7, 1152)):
        widths = wl.WIDTHS_14[C]
        idx = wl.idx_quota_uniform(wl.rng(6, 6), 256, 14)
        layer(f"M {hw}x{hw}", f"pointwise 1x1 c->c (full {C})", "uniform", 256, hw * hw, C, C, widths, widths, idx, act=1)
    # config 1: fp32 single layer
    if not want("cfg1", "fp32 linear", "iid"):
        return
    c1 = wl.config1()
    x, W = torch.from_numpy(c1["x"]).to(dev), torch.from_numpy(c1["W"]).to(dev)
    y = torch.zeros(64, 1, 256, device=dev)
    r = dsn.make_routing(64, 4, ints(np.zeros(4)), ints(np.zeros(5)), ints(np.zeros(64)), ints(np.zeros(64)))
    dsn.dsn_route(ctx, ints(c1["idx"]), 64, 4, r)
    d = dsn.make_linear_desc(dsn.F32, 1, 256, 256, c1["k_in"], c1["k_out"], W)
    us = graph_time(lambda i: dsn.dsn_sliced_linear(ctx, d, r, x, y), 8)
    fl = 2 * dsn.dsn_executed_macs(np.bincount(c1["idx"], minlength=4).tolist(), 1, c1["k_in"], c1["k_out"], 1)
    print(f"| cfg1 | fp32 linear 256x256, B=64 | iid | {us:.1f} | {fl / us / 1e6:.3f} | - | launch latency | - | - | {64 / us * 1e6:.0f} |")

# --------------------------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="dsn", choices=["dsn", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--table", action="store_true", help="print per-layer markdown rows for every configuration")
    ap.add_argument("--no-graph", action="store_true", help="time direct API calls instead of a CUDA-graph replay (for profilers)")
    ap.add_argument("--table-filter", default=None, help="with --table: only rows whose 'config layer routing' text matches this regular expression")
    ap.add_argument("--table-batch-div", type=int, default=1, help="with --table: divide every batch size by this (small cases for profilers)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    if args.table:
        run_table(args)
        return

    import torch
    from paper_2109_10060_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    import paper_2109_10060_b200 as dsn
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    ctx = dsn.Context(local_rank)
    peaks = load_peaks()

    wlk = make_workload(args.workload, dsn, torch, dev, args.batch)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        wlk.step(ctx, i)
    barrier()
    code, detail = ctx.get_status()
    if code != 0:
        raise SystemExit(f"device status {code} ({dsn.dsn_strerror(code)}) detail {detail}")
    counts = wlk.histogram()

    # The timed steps replay a CUDA graph that holds one step per rotating buffer set, so that the
    # host's launch work stays out of the device timeline.  Falls back to direct calls if capture fails.
    side = torch.cuda.Stream()
    graph, graphed = None, False
    try:
        if args.no_graph:
            raise RuntimeError("disabled by --no-graph")
        with torch.cuda.stream(side):
            wlk.step(ctx, 0)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(wlk.copies):
                wlk.step(ctx, i)
        graph.replay()
        torch.cuda.synchronize()
        graphed = True
    except Exception as exc:  # noqa: BLE001
        sys.stderr.write(f"graph capture unavailable ({exc}); timing direct calls\n")

    def run_steps(n):
        if graphed:
            for _ in range(n // wlk.copies):
                graph.replay()
            for i in range(n % wlk.copies):
                wlk.step(ctx, i)
        else:
            for i in range(n):
                wlk.step(ctx, i)

    run_steps(wlk.copies * 2)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    run_steps(args.steps)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)

    # per-kernel durations: each step of the path (same kernels, one C call each) captured as its own
    # graph over the rotating buffers and replayed back to back
    acc = {}
    marks = []
    wlk.decomposed_step(ctx, 0, lambda n: marks.append(n))
    torch.cuda.synchronize()
    part_names = marks[1:]
    for pi, pname in enumerate(part_names):
        try:
            if args.no_graph:
                raise RuntimeError("disabled by --no-graph")
            gpart = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gpart, stream=side):
                for i in range(wlk.copies):
                    wlk.decomposed_part(ctx, i, pi)
            gpart.replay()
            torch.cuda.synchronize()
            reps = 20
            e0.record(stream)
            for _ in range(reps):
                gpart.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            acc[pname] = [e0.elapsed_time(e1) / (reps * wlk.copies)]
        except Exception as exc:  # noqa: BLE001
            sys.stderr.write(f"per-kernel graph for {pname} unavailable ({exc})\n")
    if not acc:  # no graphs: direct calls with an event after each (includes launch gaps)
        for i in range(13):
            evs = []
            def mark(n):
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(stream)
                evs.append((n, ev))
            wlk.decomposed_step(ctx, i, mark)
            torch.cuda.synchronize()
            if i >= 3:
                for (n0, a), (n1, b) in zip(evs[:-1], evs[1:]):
                    acc.setdefault(n1, []).append(a.elapsed_time(b))
    wlk.decomposed_step(ctx, 0, lambda n: None)   # leave the routing arrays consistent
    torch.cuda.synchronize()
    clocks = sampler.stop()

    # end to end: batch starts and ends in pinned host memory; upload, compute and download overlap
    hx, hy = wlk.e2e_io()
    streams = (torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream())
    events = [tuple(torch.cuda.Event() for _ in range(3)) for _ in range(wlk.copies)]
    for evs in events:
        evs[2].record(stream)
    torch.cuda.synchronize()
    wlk.e2e_pipeline(ctx, hx, hy, 2 * wlk.copies, streams, events)
    barrier()
    e2e_steps = min(args.steps, 40)
    e0.record(stream)
    for st in streams:
        st.wait_event(e0)
    wlk.e2e_pipeline(ctx, hx, hy, e2e_steps, streams, events)
    for st in streams:
        ev = torch.cuda.Event()
        ev.record(st)
        stream.wait_event(ev)
    e1.record(stream)
    barrier()
    ms_e2e = e0.elapsed_time(e1) / e2e_steps
    code, detail = ctx.get_status()
    if code != 0:
        raise SystemExit(f"device status {code} ({dsn.dsn_strerror(code)}) detail {detail}")

    from paper_2109_10060_b200.sharding import max_over_ranks
    t = max_over_ranks(torch.tensor([ms_total], dtype=torch.float64, device=dev), dist if world > 1 else None)
    t2 = max_over_ranks(torch.tensor([ms_e2e], dtype=torch.float64, device=dev), dist if world > 1 else None)
    ms_step = float(t.item()) / args.steps
    ms_e2e = float(t2.item())
    flops = wlk.exec_flops(counts)
    value = world * flops / (ms_step * 1e-3) / 1e12
    e2e_value = world * flops / (ms_e2e * 1e-3) / 1e12

    if "route+gemm_chain" in acc and "route" in acc:
        gemm_ms = float(np.mean(acc["route+gemm_chain"])) - float(np.mean(acc["route"]))
        gemm_kernel = "gemm_bf16_chain_kernel (1 launch per step: conv1, conv2 and conv3 of every sample on one CTA pair)"
    else:
        gemm_ms = sum(float(np.mean(v)) for k, v in acc.items() if k.startswith("gemm:"))
        gemm_kernel = "gemm_bf16_pair_kernel (3 launches per step: conv1, conv2, conv3)"
    gemm_bytes = wlk.gemm_bytes(counts)
    achieved = gemm_bytes / (gemm_ms * 1e-3) / 1e9
    per_kernel = {k: round(float(np.mean(v)) * 1e3, 2) for k, v in acc.items()}
    roofline = {"bound": "hbm", "kernel": gemm_kernel,
                "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "peak_source": peaks["source"] + " copy bandwidth, burst",
                # dram__bytes_read + dram__bytes_write of one launch of this kernel on this workload (ncu capture
                # summarised under profiles/; to be re-taken, or set to None, whenever the kernel changes)
                "traffic": CHAIN_CFG2_DRAM_BYTES if (gemm_kernel.startswith("gemm_bf16_chain") and args.workload == "cfg2"
                                                     and args.batch in (None, 128)) else None,
                "algorithmic_bytes_per_step": gemm_bytes, "us_per_step": round(gemm_ms * 1e3, 2),
                "executed_tflops": flops / (gemm_ms * 1e-3) / 1e12,
                "frac_of_bf16_peak_burst": flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}

    if rank != 0:
        return
    out = {
        "metric": "sliced_gemm_executed_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{wlk.name}: batch {wlk.B} per GPU, gate-driven routing" if wlk.gate_driven
                   else f"{wlk.name}: batch {wlk.B} per GPU, routing {wlk.cfg['routing']}",
                   "path": "gate -> route -> 1x1 -> 3x3 -> 1x1 -> input order (dsn_layer_forward)",
                   "l2": f"inputs and outputs rotate over {wlk.copies} buffers (> 126 MB L2)",
                   "launch": "CUDA graph replay of the public-API step" if graphed else "direct calls",
                   "routing_histogram": counts.tolist(), "parallelism": f"batch shards x{world}, no collective"},
        "samples_per_s": world * wlk.B / (ms_step * 1e-3),
        "pct_bf16_peak_burst": 100 * value / world / peaks["bf16_tflops"],
        "pct_bf16_peak_nominal": 100 * value / world / NOMINAL_BF16_TFLOPS,
        "kernel_us": per_kernel,
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": int(hx.numel() * 2),
                "d2h_bytes_per_step": int(hy.numel() * 2), "ms_per_step": ms_e2e,
                "how": "dsn_layer_forward per step; upload, compute and download pipelined on three streams"},
        "gpu_launches": wlk.kernels_per_step * args.steps,
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        n = wlk.B
        f_cpu, dt = wlk.oracle_sample(n)
        out["cpu_baseline"] = {"value": f_cpu / dt / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
                               "sample": f"{n} of {wlk.B} samples, gate + route + bottleneck chain, fp64 numpy (threaded BLAS), {dt:.1f} s wall"}
    print(json.dumps(out))


if __name__ == "__main__":
    main()
