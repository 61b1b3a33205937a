#!/usr/bin/env python
"""Benchmark of the dynamic-weight-slicing hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: gate (average pool,
FC-ReLU-FC, arg-max) -> routing (stable grouping) -> the block's sliced grouped GEMMs (and, for a
ViT block, the attention core between QKV and the projection) -> outputs in input order.

Default workload (--workload cfg5): serving-scale ViT-B-width dynamic block, bf16, 1024 samples x 197
tokens, embed 768, 12 heads, MLP 3072, 8 diagonal paths, quota-uniform routing: gate, then
dsn_layer_forward(QKV -> attention -> proj), then dsn_layer_forward(fc1-GELU -> fc2) on the same
routing.  Other workloads: cfg2, cfg3, cfg4-stage{1..4}[-uniform], M (DS-MBNet depthwise + pointwise).

Prints ONE JSON line (see --help).  `value` is executed TFLOP/s of the whole step (2 x multiply-adds
of the contractions actually run, divided by the step time, gate and routing included), inputs
resident in HBM.  `e2e` is the same metric with the batch starting and ending in pinned host memory.
`roofline` describes the dominant grouped-GEMM launch, `cpu_baseline` the fp64 CPU oracle on a bounded
sample, `per_config` holds the per-layer rows of every configuration.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
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
MIN_TIMED_SECONDS = 0.2           # the timed region lasts at least this long whatever --steps says


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


# --------------------------------------------------------------------------------------------- helpers
def kernel_source_digest(files):
    """sha256 over the named kernel sources (relative to the package's csrc folder)."""
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2109_10060_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def recorded_traffic(kernel, workload):
    """DRAM bytes per launch from an ncu summary under profiles/, or None.  A summary carries a line
    `bench-traffic: kernel=<k> workload=<w> bytes=<n> sources=<a.cu,b.cuh> sha256=<digest>`; the figure is
    used only while the digest of those sources is unchanged (a changed kernel invalidates its counters)."""
    pdir = os.path.join(ROOT, "profiles")
    if not os.path.isdir(pdir):
        return None
    for name in sorted(os.listdir(pdir)):
        try:
            text = open(os.path.join(pdir, name)).read()
        except OSError:
            continue
        for m in re.finditer(r"bench-traffic: kernel=(\S+) workload=(\S+) bytes=(\d+) sources=(\S+) sha256=(\w+)", text):
            if m.group(1) == kernel and m.group(2) == workload:
                try:
                    if kernel_source_digest(m.group(4).split(",")) == m.group(5):
                        return int(m.group(3))
                except OSError:
                    pass
    return None


class GraphTimer:
    """Times a sequence of API calls on the device: one CUDA graph holding `nbuf` calls (one per rotating
    buffer set), replayed until the timed region is long enough; CUDA events on the replaying stream."""

    def __init__(self, torch, use_graph=True):
        self.torch = torch
        self.use_graph = use_graph
        self.side = torch.cuda.Stream()

    def time_us(self, call, nbuf, min_seconds=0.05, max_replays=4000):
        t = self.torch
        with t.cuda.stream(self.side):
            call(0)
        t.cuda.synchronize()
        e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
        if not self.use_graph:   # direct calls: one untimed pass over the buffers, then timed passes
            with t.cuda.stream(self.side):
                for i in range(nbuf):
                    call(i)
                e0.record(self.side)
                for i in range(2 * nbuf):
                    call(i)
                e1.record(self.side)
            t.cuda.synchronize()
            return e0.elapsed_time(e1) / (2 * nbuf) * 1e3
        g = t.cuda.CUDAGraph()
        with t.cuda.graph(g, stream=self.side):
            for i in range(nbuf):
                call(i)
        cur = t.cuda.current_stream()
        for _ in range(3):
            g.replay()
        e0.record(cur)
        g.replay()
        e1.record(cur)
        t.cuda.synchronize()
        once = max(e0.elapsed_time(e1) * 1e-3, 1e-6)
        reps = int(min(max_replays, max(3, math.ceil(min_seconds / once))))
        e0.record(cur)
        for _ in range(reps):
            g.replay()
        e1.record(cur)
        t.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * nbuf) * 1e3


def burst_time_us(torch, call, nbuf, launches=8):
    """The launch timed alone, the way the burst peaks were measured: after an idle pause (clocks back at
    their maximum), one untimed call, then the best of a few single calls, each bracketed by CUDA events."""
    torch.cuda.synchronize()
    time.sleep(0.25)
    call(0)
    best = float("inf")
    for i in range(launches):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        call((i + 1) % nbuf)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) * 1e3)
    return best


def gemm_algorithmic_bytes(counts, R, k_in, k_out, K=1):
    """Sliced input read once, sliced output written once, every used weight slice read once (bf16)."""
    return sum(2 * (int(n) * R * (k_in[t] + k_out[t]) + k_in[t] * k_out[t] * K * K) for t, n in enumerate(counts) if n)


# --------------------------------------------------------------------------------------------- workloads
class Workload:
    """What the timing code needs from a workload."""
    gate_driven = False

    def x_buffers(self):
        return self.xs

    def y_buffers(self):
        return self.ys

    def e2e_io(self):
        t = self.torch
        hx = t.from_numpy(self.x_host_bits.copy()).pin_memory()
        hy = t.empty(self.ys[0].numel(), dtype=t.int16).pin_memory()
        return hx, hy

    def e2e_pipeline(self, ctx, hx, hy, n, streams, events):
        """n steps with the batch starting and ending in pinned host memory: the upload of step i+1, the
        compute of step i and the download of step i-1 run on three streams over the rotating buffer sets."""
        t = self.torch
        s_up, s_run, s_down = streams
        for i in range(n):
            k = i % len(events)
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


class Bottleneck(Workload):
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
        self.slices = [("conv1_1x1", full, self.widths, 1), ("conv2_3x3", self.widths, self.widths, 3),
                       ("conv3_1x1", self.widths, full, 1)]
        mk = dsn.make_conv_desc
        self.layers = [mk(dsn.BF16, H, Wd, 1, 0, C, Ci, full, self.widths, self.W1, act=dsn.ACT_RELU),
                       mk(dsn.BF16, H, Wd, 3, 1, Ci, Ci, self.widths, self.widths, self.W2, act=dsn.ACT_RELU),
                       mk(dsn.BF16, H, Wd, 1, 0, Ci, C, self.widths, full, self.W3)]
        self.gW1 = torch.from_numpy(cfg["gate_W1"]).to(dev)
        self.gW2 = torch.from_numpy(cfg["gate_W2"]).to(dev)
        self.gate = dsn.make_gate_desc(dsn.BF16, B, self.R, C, self.gW1.shape[0], T, self.gW1, self.gW2)
        self.idx_given = torch.from_numpy(cfg["idx"]).to(dev)
        self.L = dsn.make_layer_desc(B, T, self.layers, self.gate if gate_driven else None)
        self.L_given = dsn.make_layer_desc(B, T, self.layers, None)
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
        # launches per step: gate = pool + hidden + score, route, then one chained launch or three GEMMs
        self.kernels_per_step = (3 if gate_driven else 0) + 1 + (1 if self.chained else 3)
        self.name = cfg["name"]
        self.path = "gate -> route -> 1x1 -> 3x3 -> 1x1 -> input order (one dsn_layer_forward call)"
        self.routing_name = "gate-driven" if gate_driven else cfg["routing"]
        self.flops_note = "2 x multiply-adds of the three sliced convolutions at the routing histogram"

    def step(self, ctx, i):
        k = i % self.copies
        self.dsn.dsn_layer_forward(ctx, self.L, self.xs[k], None if self.gate_driven else self.idx_given, self.ys[k],
                                   self.ws, idx_out=self.idx_out if self.gate_driven else None)

    def histogram(self):
        return np.bincount(self.idx_out.cpu().numpy() if self.gate_driven else self.cfg["idx"], minlength=self.T)

    def parts(self, counts):
        """(name, call(ctx, k), flops, algorithmic bytes, kind) of every step of the path as its own C call."""
        d, c = self.dsn, counts.tolist()
        src = self.idx_out if self.gate_driven else self.idx_given
        out = []
        if self.gate_driven:
            out.append(("gate", lambda ctx, k: d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws),
                        0, 2 * self.B * self.R * self.C, "hbm"))
        out.append(("route", lambda ctx, k: d.dsn_route(ctx, src, self.B, self.T, self.routing), 0, 20 * self.B, "latency"))
        fl = [2 * d.dsn_executed_macs(c, self.R, ki, ko, K) for _, ki, ko, K in self.slices]
        by = [gemm_algorithmic_bytes(c, self.R, ki, ko, K) for _, ki, ko, K in self.slices]
        if self.chained:
            # the step's own launch: route + the chained GEMM launch on given indices (one API call)
            out.append(("route+gemm_chain", lambda ctx, k: d.dsn_layer_forward(ctx, self.L_given, self.xs[k], src, self.ys[k], self.ws),
                        sum(fl), sum(by), "chain"))
        calls = [lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[0], self.routing, self.xs[k], self.t1),
                 lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[1], self.routing, self.t1, self.t2),
                 lambda ctx, k: d.dsn_sliced_conv(ctx, self.dec_layers[2], self.routing, self.t2, self.ys[k])]
        for (lname, _, _, _), call, f, b in zip(self.slices, calls, fl, by):
            out.append(("gemm:" + lname, call, f, b, "gemm"))
        return out

    def exec_flops(self, counts):
        return sum(2 * self.dsn.dsn_executed_macs(counts.tolist(), self.R, ki, ko, K) for _, ki, ko, K in self.slices)

    def oracle_run(self, samples, idx_given=None):
        """Runs the fp64 oracle on the given samples (gate + route + bottleneck chain); returns executed flops."""
        from oracle import dsn_oracle as O
        cfg = self.cfg
        x = cfg["x"][samples]
        idx, _, _ = O.gate(x.reshape(len(samples), self.R, self.C), cfg["gate_W1"], cfg["gate_W2"])
        if not self.gate_driven:
            idx = cfg["idx"][samples]
        O.route(idx, self.T)
        O.bottleneck(x, cfg["W1"], cfg["W2"], cfg["W3"], idx, self.widths, mirror_bf16=True)
        return sum(2 * O.executed_macs(idx, self.R, ki, ko, K) for _, ki, ko, K in self.slices)

    def oracle_samples(self, n, offset=0):
        return [(offset * n + j) % self.B for j in range(n)]

    oracle_what = "gate + route + bottleneck chain, fp64 numpy (threaded BLAS)"


class ViTBlock(Workload):
    """DS-ViT-style dynamic transformer block (configs 3 and 5): gate on the mean token, then one
    dsn_layer_forward call whose five elements inherit one routing: QKV -> attention core -> proj ->
    fc1(GELU) -> fc2.  routing = "gate" lets the gate's own choice route the batch;
    any other name routes by the given seeded draw (the gate still runs and its choice is recorded)."""

    def __init__(self, dsn, torch, dev, cfg, routing, copies=None):
        import dsn_workloads as wl
        self.dsn, self.torch, self.dev, self.cfg = dsn, torch, dev, cfg
        B, R, De, H, Dh, Dm, T, paths = (cfg["B"], cfg["R"], cfg["D_e"], cfg["H"], cfg["D_h"], cfg["D_mlp"], cfg["T"],
                                         cfg["paths"])
        self.B, self.R, self.De, self.H, self.Dh, self.Dm, self.T, self.paths = B, R, De, H, Dh, Dm, T, paths
        self.gate_driven = routing == "gate"
        self.heads = [p[1] for p in paths]
        up = lambda a: torch.from_numpy(wl.bf16_bits(np.ascontiguousarray(a)).view(np.int16)).to(dev).view(torch.bfloat16).reshape(a.shape)
        self.x_host_bits = wl.bf16_bits(cfg["x"]).view(np.int16)
        x_bytes = self.x_host_bits.nbytes
        # the block input alone is larger than L2 for the serving-scale config; smaller batches rotate buffer sets
        self.copies = copies or max(2, -(-2 * L2_BYTES // (2 * x_bytes)) + 1)   # two sets at least: the host pipeline overlaps them
        self.xs = [torch.from_numpy(self.x_host_bits).to(dev).view(torch.bfloat16).reshape(B, R, De) for _ in range(self.copies)]
        self.ys = [torch.zeros(B, R, De, dtype=torch.bfloat16, device=dev) for _ in range(self.copies)]
        self.Wqkv = up(wl.pack_qkv_head_major(cfg["Wq"], cfg["Wk"], cfg["Wv"], Dh))
        self.Wproj, self.Wfc1, self.Wfc2 = up(cfg["Wproj"]), up(cfg["Wfc1"]), up(cfg["Wfc2"])
        sl = {n: wl.vit_layer_slices(paths, Dh, n) for n in ("qkv", "proj", "fc1", "fc2")}
        self.sl = sl
        ml, ma = dsn.make_linear_desc, dsn.make_attention_desc
        HD = H * Dh
        self.att_layers = [ml(dsn.BF16, R, De, 3 * HD, *sl["qkv"], self.Wqkv), ma(R, H, Dh, self.heads),
                           ml(dsn.BF16, R, HD, De, *sl["proj"], self.Wproj)]
        self.mlp_layers = [ml(dsn.BF16, R, De, Dm, *sl["fc1"], self.Wfc1, act=dsn.ACT_GELU),
                           ml(dsn.BF16, R, Dm, De, *sl["fc2"], self.Wfc2)]
        self.gW1 = torch.from_numpy(cfg["gate_W1"]).to(dev)
        self.gW2 = torch.from_numpy(cfg["gate_W2"]).to(dev)
        self.gate = dsn.make_gate_desc(dsn.BF16, B, R, De, self.gW1.shape[0], T, self.gW1, self.gW2)
        self.L = dsn.make_layer_desc(B, T, self.att_layers + self.mlp_layers, self.gate if self.gate_driven else None)
        self.ws = torch.empty(dsn.dsn_layer_workspace_bytes(self.L), dtype=torch.uint8, device=dev)
        self.gate_ws = torch.empty(dsn.dsn_gate_workspace_bytes(self.gate), dtype=torch.uint8, device=dev)
        self.idx_given = torch.from_numpy(np.ascontiguousarray(cfg["idx"], dtype=np.int32)).to(dev)
        self.idx_out = torch.zeros(B, dtype=torch.int32, device=dev)
        # decomposed form for per-kernel timing: the same kernels, one C call each, on buffers of their own
        ints = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
        self.routing = dsn.make_routing(B, T, ints(T), ints(T + 1), ints(B), ints(B))
        self.t_qkv = torch.zeros(B, R, 3 * HD, dtype=torch.bfloat16, device=dev)
        self.t_att = torch.zeros(B, R, HD, dtype=torch.bfloat16, device=dev)
        self.t_h = torch.zeros(B, R, De, dtype=torch.bfloat16, device=dev)
        self.t_hid = torch.zeros(B, R, Dm, dtype=torch.bfloat16, device=dev)
        G, I = dsn.GROUPED, dsn.INPUT_ORDER
        self.dec = {
            "qkv": ml(dsn.BF16, R, De, 3 * HD, *sl["qkv"], self.Wqkv, in_order=I, out_order=G),
            "attention": ma(R, H, Dh, self.heads, order=G),
            "proj": ml(dsn.BF16, R, HD, De, *sl["proj"], self.Wproj, in_order=G, out_order=G),
            "fc1": ml(dsn.BF16, R, De, Dm, *sl["fc1"], self.Wfc1, act=dsn.ACT_GELU, in_order=G, out_order=G),
            "fc2": ml(dsn.BF16, R, Dm, De, *sl["fc2"], self.Wfc2, in_order=G, out_order=I)}
        # launches per step: gate (pool, hidden, scores), route, five layers
        self.kernels_per_step = 3 + 1 + 5
        self.name = cfg["name"]
        self.routing_name = "gate-driven" if self.gate_driven else cfg["routing"]
        self.path = ("gate -> route -> QKV -> attention core -> proj -> fc1(GELU) -> fc2 -> input order: "
                     + ("one dsn_layer_forward call, all five elements under the gate's one decision" if self.gate_driven
                        else "dsn_gate, then one dsn_layer_forward call on the given routing (all five elements under one decision)"))
        self.flops_note = ("2 x multiply-adds of QKV, proj, fc1, fc2 at the routing histogram + 4 N^2 D_h per executed "
                           "head for the attention core (QK^T and PV)")

    def step(self, ctx, i):
        k, d = i % self.copies, self.dsn
        if self.gate_driven:
            d.dsn_layer_forward(ctx, self.L, self.xs[k], None, self.ys[k], self.ws, idx_out=self.idx_out)
        else:
            d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws)
            d.dsn_layer_forward(ctx, self.L, self.xs[k], self.idx_given, self.ys[k], self.ws)

    def histogram(self):
        return np.bincount(self.idx_out.cpu().numpy() if self.gate_driven else self.cfg["idx"], minlength=self.T)

    def attention_flops(self, counts):
        return sum(4.0 * self.R * self.R * self.Dh * self.heads[t] * int(n) for t, n in enumerate(counts))

    def parts(self, counts):
        d, c = self.dsn, counts.tolist()
        src = self.idx_out if self.gate_driven else self.idx_given
        fl = {n: 2 * d.dsn_executed_macs(c, self.R, *self.sl[n], 1) for n in self.sl}
        by = {n: gemm_algorithmic_bytes(c, self.R, *self.sl[n]) for n in self.sl}
        att_bytes = sum(2.0 * self.R * 4 * self.Dh * self.heads[t] * int(n) for t, n in enumerate(c))
        r = self.routing
        return [
            ("gate", lambda ctx, k: d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws), 0,
             2 * self.B * self.R * self.De, "hbm"),
            ("route", lambda ctx, k: d.dsn_route(ctx, src, self.B, self.T, r), 0, 20 * self.B, "latency"),
            ("gemm:qkv", lambda ctx, k: d.dsn_sliced_linear(ctx, self.dec["qkv"], r, self.xs[k], self.t_qkv), fl["qkv"], by["qkv"], "gemm"),
            ("attention", lambda ctx, k: d.dsn_sliced_attention(ctx, self.dec["attention"], r, self.t_qkv, self.t_att),
             self.attention_flops(c), att_bytes, "attention"),
            ("gemm:proj", lambda ctx, k: d.dsn_sliced_linear(ctx, self.dec["proj"], r, self.t_att, self.t_h), fl["proj"], by["proj"], "gemm"),
            ("gemm:fc1", lambda ctx, k: d.dsn_sliced_linear(ctx, self.dec["fc1"], r, self.t_h, self.t_hid), fl["fc1"], by["fc1"], "gemm"),
            ("gemm:fc2", lambda ctx, k: d.dsn_sliced_linear(ctx, self.dec["fc2"], r, self.t_hid, self.ys[k]), fl["fc2"], by["fc2"], "gemm"),
        ]

    def exec_flops(self, counts):
        c = counts.tolist()
        return sum(2 * self.dsn.dsn_executed_macs(c, self.R, *self.sl[n], 1) for n in self.sl) + self.attention_flops(c)

    def oracle_run(self, samples, idx_given=None):
        from oracle import dsn_oracle as O
        cfg = self.cfg
        x = cfg["x"][samples]
        idx, _, _ = O.gate(x, cfg["gate_W1"], cfg["gate_W2"])
        if not self.gate_driven:
            idx = np.asarray(cfg["idx"])[samples]
        O.route(idx, self.T)
        h = O.vit_attention_half(x, cfg["Wq"], cfg["Wk"], cfg["Wv"], cfg["Wproj"], idx, self.paths, self.Dh)[4]
        O.vit_mlp(np.nan_to_num(h), cfg["Wfc1"], cfg["Wfc2"], idx, self.paths, mirror_bf16=True)
        counts = np.bincount(idx, minlength=self.T)
        return (sum(2 * O.executed_macs(idx, self.R, *self.sl[n]) for n in self.sl) + self.attention_flops(counts))

    def oracle_samples(self, n, offset=0):
        """n samples spread over the paths in use (one per path first)."""
        idx = np.asarray(self.cfg["idx"])
        order = np.argsort(idx, kind="stable")
        firsts = [int(order[np.searchsorted(idx[order], t)]) for t in np.unique(idx)]
        pick = [(firsts[j % len(firsts)] + offset * 7 + (j // len(firsts)) * 13) % self.B for j in range(n)]
        return pick

    oracle_what = "gate + route + QKV + attention + proj + fc1(GELU) + fc2, fp64 numpy (threaded BLAS)"


class MobileNetBlock(Workload):
    """DS-MBNet separable block (supplementary workload): gate, route, slice-able depthwise 3x3 on the c_t
    leading channels (ReLU), pointwise 1x1 c_t -> c_t (ReLU), outputs in input order."""

    def __init__(self, dsn, torch, dev, cfg, copies=None):
        import dsn_workloads as wl
        self.dsn, self.torch, self.dev, self.cfg = dsn, torch, dev, cfg
        B, H, Wd, C, K, T = cfg["B"], cfg["H"], cfg["W"], cfg["C"], cfg["K"], cfg["T"]
        self._host(cfg)
        up = lambda a: torch.from_numpy(wl.bf16_bits(np.ascontiguousarray(a)).view(np.int16)).to(dev).view(torch.bfloat16).reshape(a.shape)
        self.x_host_bits = wl.bf16_bits(cfg["x"]).view(np.int16)
        self.copies = copies or -(-2 * L2_BYTES // (2 * self.x_host_bits.nbytes)) + 1
        self.xs = [torch.from_numpy(self.x_host_bits).to(dev).view(torch.bfloat16).reshape(B, H, Wd, C) for _ in range(self.copies)]
        self.ys = [torch.zeros(B, H, Wd, C, dtype=torch.bfloat16, device=dev) for _ in range(self.copies)]
        self.Wdw = up(np.transpose(cfg["Wdw"], (1, 2, 0)))
        self.Wpw = up(cfg["Wpw"].reshape(C, C))
        w = self.widths
        self.dw = dsn.make_depthwise_desc(H, Wd, K, 1, C, w, [K] * T, self.Wdw, act=dsn.ACT_RELU,
                                          in_order=dsn.INPUT_ORDER, out_order=dsn.GROUPED)
        self.pw = dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, C, w, w, self.Wpw, act=dsn.ACT_RELU,
                                     in_order=dsn.GROUPED, out_order=dsn.INPUT_ORDER)
        # the step: one dsn_layer_forward call (depthwise, then pointwise; one kernel under DSN_DWPW=fused)
        self.L = dsn.make_layer_desc(B, T, [dsn.make_depthwise_desc(H, Wd, K, 1, C, w, [K] * T, self.Wdw, act=dsn.ACT_RELU),
                                            dsn.make_conv_desc(dsn.BF16, H, Wd, 1, 0, C, C, w, w, self.Wpw, act=dsn.ACT_RELU)], None)
        self.ws = torch.empty(dsn.dsn_layer_workspace_bytes(self.L), dtype=torch.uint8, device=dev)
        self.gW1 = torch.from_numpy(cfg["gate_W1"]).to(dev)
        self.gW2 = torch.from_numpy(cfg["gate_W2"]).to(dev)
        self.gate = dsn.make_gate_desc(dsn.BF16, B, self.R, C, self.gW1.shape[0], T, self.gW1, self.gW2)
        self.gate_ws = torch.empty(dsn.dsn_gate_workspace_bytes(self.gate), dtype=torch.uint8, device=dev)
        self.idx_given = torch.from_numpy(np.ascontiguousarray(cfg["idx"], dtype=np.int32)).to(dev)
        self.idx_out = torch.zeros(B, dtype=torch.int32, device=dev)
        ints = lambda n: torch.zeros(n, dtype=torch.int32, device=dev)
        self.routing = dsn.make_routing(B, T, ints(T), ints(T + 1), ints(B), ints(B))
        self.t_dw = torch.zeros(B, H, Wd, C, dtype=torch.bfloat16, device=dev)
        self.kernels_per_step = 3 + 1 + (1 if os.environ.get("DSN_DWPW") == "fused" else 2)
        self.name = cfg["name"]
        self.routing_name = cfg["routing"]
        self.path = ("gate -> route -> depthwise 3x3 (ReLU) -> pointwise 1x1 (ReLU) -> input order: dsn_gate, then one "
                     "dsn_layer_forward call on the given routing")
        self.flops_note = "2 x multiply-adds of the depthwise (9 c_t per pixel) and pointwise (c_t^2 per pixel) layers"

    def _host(self, cfg):
        self.cfg = cfg
        self.B, self.R, self.C, self.K, self.T, self.widths = cfg["B"], cfg["H"] * cfg["W"], cfg["C"], cfg["K"], cfg["T"], cfg["widths"]

    @classmethod
    def host_only(cls, cfg):
        w = cls.__new__(cls)
        w._host(cfg)
        return w

    def step(self, ctx, i):
        k, d = i % self.copies, self.dsn
        d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws)
        d.dsn_layer_forward(ctx, self.L, self.xs[k], self.idx_given, self.ys[k], self.ws)

    def histogram(self):
        return np.bincount(self.cfg["idx"], minlength=self.T)

    def _flops(self, counts):
        dw = sum(2.0 * self.R * self.K * self.K * self.widths[t] * int(n) for t, n in enumerate(counts))
        pw = sum(2.0 * self.R * self.widths[t] ** 2 * int(n) for t, n in enumerate(counts))
        return dw, pw

    def parts(self, counts):
        d, c, r, w = self.dsn, counts.tolist(), self.routing, self.widths
        dwf, pwf = self._flops(c)
        dw_bytes = sum(2.0 * 2 * self.R * w[t] * int(n) for t, n in enumerate(c))
        return [
            ("gate", lambda ctx, k: d.dsn_gate(ctx, self.gate, self.xs[k], self.idx_out, None, self.gate_ws), 0,
             2 * self.B * self.R * self.C, "hbm"),
            ("route", lambda ctx, k: d.dsn_route(ctx, self.idx_given, self.B, self.T, r), 0, 20 * self.B, "latency"),
            ("route+depthwise+pointwise (the step's dsn_layer_forward call)",
             lambda ctx, k: d.dsn_layer_forward(ctx, self.L, self.xs[k], self.idx_given, self.ys[k], self.ws),
             dwf + pwf, dw_bytes + gemm_algorithmic_bytes(c, self.R, w, w), "other"),
            ("depthwise", lambda ctx, k: d.dsn_sliced_depthwise(ctx, self.dw, r, self.xs[k], self.t_dw), dwf, dw_bytes, "hbm"),
            ("gemm:pointwise", lambda ctx, k: d.dsn_sliced_conv(ctx, self.pw, r, self.t_dw, self.ys[k]), pwf,
             gemm_algorithmic_bytes(c, self.R, w, w), "gemm"),
        ]

    def exec_flops(self, counts):
        return sum(self._flops(counts.tolist()))

    def oracle_run(self, samples, idx_given=None):
        from oracle import dsn_oracle as O
        cfg = self.cfg
        x = cfg["x"][samples]
        O.gate(x.reshape(len(samples), self.R, self.C), cfg["gate_W1"], cfg["gate_W2"])
        idx = np.asarray(cfg["idx"])[samples]
        O.route(idx, self.T)
        t = O.round_bf16(O.sliced_depthwise(x, cfg["Wdw"], idx, self.widths, [self.K] * self.T, act=O.ACT_RELU, fill=0.0))
        O.round_bf16(O.sliced_conv(t, cfg["Wpw"], idx, self.widths, self.widths, 0, act=O.ACT_RELU))
        return sum(self._flops(np.bincount(idx, minlength=self.T).tolist()))

    def oracle_samples(self, n, offset=0):
        return [(offset * n + j) % self.B for j in range(n)]

    oracle_what = "gate + route + depthwise 3x3 + pointwise 1x1, fp64 numpy"


WORKLOADS = ("cfg2", "cfg3", "cfg4-stage1", "cfg4-stage2", "cfg4-stage3", "cfg4-stage4", "cfg4-stage1-uniform",
             "cfg4-stage2-uniform", "cfg4-stage3-uniform", "cfg4-stage4-uniform", "cfg5", "M")


def make_workload(name, dsn, torch, dev, batch=None, routing=None):
    import dsn_workloads as wl
    vit_routing = {"uniform": dict(routing="uniform"), "zipf": dict(routing="zipf"), "gate": dict(routing="uniform"),
                   "one0": dict(routing="one", one_path=0), "one7": dict(routing="one", one_path=7)}
    if name == "cfg2":
        return Bottleneck(dsn, torch, dev, wl.config2(B=batch or 128), gate_driven=routing in (None, "gate"))
    if name.startswith("cfg4-stage"):
        stage = int(name[len("cfg4-stage")])
        r = "uniform" if name.endswith("uniform") else "skewed"
        return Bottleneck(dsn, torch, dev, wl.config4(stage, B=batch or 256, routing=r), gate_driven=False)
    if name in ("cfg3", "cfg5"):
        r = routing or "uniform"
        if r not in vit_routing:
            raise SystemExit(f"unknown routing {r} for {name}")
        kw = dict(vit_routing[r])
        if name == "cfg3":
            kw.pop("one_path", None)
            cfg = wl.config3(B=batch or 256, routing=kw["routing"])
        else:
            cfg = wl.config5(B=batch or 1024, **kw)
        return ViTBlock(dsn, torch, dev, cfg, routing=r)
    if name == "M":
        return MobileNetBlock(dsn, torch, dev, wl.mobilenet_block(B=batch or 256))
    raise SystemExit(f"unknown workload {name}; choose from {', '.join(WORKLOADS)}")


def workload_title(name):
    return {"cfg2": "cfg2 ResNet-50 stage-3 dynamic bottleneck, bf16 NHWC, 14x14, 1024->w->w->1024, 14 inner widths",
            "cfg3": "cfg3 DS-ViT-style block, bf16, 197 tokens, embed 384, 6 heads, MLP 1536, 48 paths",
            "cfg5": "cfg5 serving-scale ViT-B-width dynamic block, bf16, 197 tokens, embed 768, 12 heads, MLP 3072, 8 diagonal paths",
            "M": "M DS-MBNet separable block, bf16 NHWC, 14x14, depthwise 3x3 + pointwise 1x1, 14 widths 224..640"}.get(
                name, f"{name} ResNet-50 dynamic bottleneck of that stage, bf16 NHWC, 14 inner widths")


# --------------------------------------------------------------------------------------------- reference arm
class _HostOnly:
    """Stands in for the torch / library handles when only a workload's host-side data is wanted."""
    def __getattr__(self, name):
        raise RuntimeError("the reference arm runs on the host only")


def host_workload(name, batch, routing):
    """The workload object without any device allocation: only what oracle_run / oracle_samples use."""
    import dsn_workloads as wl
    if name == "cfg2" or name.startswith("cfg4-stage"):
        if name == "cfg2":
            cfg, gd = wl.config2(B=batch or 128), routing in (None, "gate")
        else:
            cfg, gd = wl.config4(int(name[len("cfg4-stage")]), B=batch or 256,
                                 routing="uniform" if name.endswith("uniform") else "skewed"), False
        w = Bottleneck.__new__(Bottleneck)
        C, T = cfg["C_outer"], cfg["T"]
        w.cfg, w.B, w.R, w.C, w.T, w.widths, w.gate_driven = cfg, cfg["B"], cfg["H"] * cfg["W"], C, T, cfg["widths"], gd
        w.slices = [("conv1_1x1", [C] * T, w.widths, 1), ("conv2_3x3", w.widths, w.widths, 3), ("conv3_1x1", w.widths, [C] * T, 1)]
        return w
    if name in ("cfg3", "cfg5"):
        r = routing or "uniform"
        kind = {"uniform": "uniform", "zipf": "zipf", "gate": "uniform", "one0": "one", "one7": "one"}[r]
        cfg = (wl.config3(B=batch or 256, routing=kind) if name == "cfg3"
               else wl.config5(B=batch or 1024, routing=kind, one_path=0 if r == "one0" else 7))
        w = ViTBlock.__new__(ViTBlock)
        w.cfg, w.B, w.R, w.Dh, w.T, w.paths = cfg, cfg["B"], cfg["R"], cfg["D_h"], cfg["T"], cfg["paths"]
        w.heads = [p[1] for p in w.paths]
        w.gate_driven = r == "gate"
        w.sl = {n: wl.vit_layer_slices(w.paths, w.Dh, n) for n in ("qkv", "proj", "fc1", "fc2")}
        return w
    if name == "M":
        return MobileNetBlock.host_only(wl.mobilenet_block(B=batch or 256))
    raise SystemExit(f"unknown workload {name}")


def run_reference(args):
    """Times the CPU oracle (the only 'reference implementation' this method has) on host cores: every
    step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = host_workload(args.workload, args.batch, args.routing)
    n = {"cfg5": 8, "cfg3": 16}.get(args.workload, 8)
    for i in range(min(args.warmup, 3)):
        w.oracle_run(w.oracle_samples(n, i))
    flops, t0 = 0, time.perf_counter()
    for i in range(args.steps):
        flops += w.oracle_run(w.oracle_samples(n, i))
    dt = time.perf_counter() - t0
    val = flops / dt / 1e12
    cores = os.cpu_count()
    print(json.dumps({
        "impl": "reference", "metric": "sliced_gemm_executed_tflops", "value": val, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_title(args.workload), "batch": w.B,
                   "routing": "gate-driven" if w.gate_driven else w.cfg["routing"],
                   "sample": f"{n} of {w.B} samples per step"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "sample": f"{n} of {w.B} samples per step, {args.steps} steps; {w.oracle_what}"},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# --------------------------------------------------------------------------------------------- per-layer rows
def collect_rows(dsn, torch, ctx, dev, peaks, timer, row_filter=None, batch_div=1, emit=None):
    """Per-layer numbers for every configuration: CUDA-graph replay over rotating buffers larger than L2,
    executed TFLOP/s and fraction of the shape's roofline bound min(measured BF16 peak, intensity x measured
    HBM bandwidth).  Returns a list of dict rows; `emit(row)` is called as each row is measured."""
    import dsn_workloads as wl
    PEAK, HBM = peaks["bf16_tflops"], peaks["hbm_gbs"]
    ints = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)
    want = (lambda *names: re.search(row_filter, " ".join(names)) is not None) if row_filter else (lambda *names: True)
    div = max(1, batch_div)
    rows = []

    def add(row):
        rows.append(row)
        if emit:
            emit(row)

    def gemm_row(cfgname, lname, rname, B, us, flops, byts, floor_util=None):
        tf = flops / us / 1e6
        bound = min(PEAK, flops / byts * HBM / 1e3)
        row = {"config": cfgname, "layer": lname, "routing": rname, "us": round(us, 1), "tflops": round(tf, 1),
               "pct_bf16_peak": round(100 * tf / PEAK, 1), "bound_tflops": round(bound), "pct_of_bound": round(100 * tf / bound),
               "gbs": round(byts / us / 1e3), "samples_per_s": round(B / us * 1e6)}
        if floor_util is not None and floor_util < 0.995:
            # a tcgen05.mma of N columns occupies the tensor pipe for max(59, N / 2) cycles (measured): narrow slices
            # cannot use more than this share of the peak, whatever the kernel does
            fb = min(bound, PEAK * floor_util)
            row["bound_with_mma_floor_tflops"] = round(fb)
            row["pct_of_bound_with_mma_floor"] = round(100 * tf / fb)
        add(row)

    def mma_floor_util(counts, R, k_in, k_out, K):
        """Share of the tensor peak the executed FLOPs can reach when every instruction of N < 118 columns still
        occupies the pipe for 59 cycles: FLOP-weighted over the slices and their n-tiles."""
        bn = 256 if max(k_out) > 128 else (128 if max(k_out) > 64 else 64)
        fl = tm = 0.0
        for t, n in enumerate(counts):
            if not n:
                continue
            for n0 in range(0, k_out[t], bn):
                cols = min(bn, k_out[t] - n0)
                n_inst = min(bn, (cols + 31) // 32 * 32)
                f = float(n) * R * k_in[t] * cols * K * K
                fl += f
                tm += f / cols * n_inst / ((n_inst / 2) / max(59.0, n_inst / 2))   # issued columns / pipe share
        return fl / tm if tm else 1.0

    def routed(B, T, idx):
        r = dsn.make_routing(B, T, ints(np.zeros(T)), ints(np.zeros(T + 1)), ints(np.zeros(B)), ints(np.zeros(B)))
        dsn.dsn_route(ctx, ints(idx), B, T, r)
        return r

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
        r = routed(B, T, idx) if group_list is None else group_list
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
        us = timer.time_us(call, nbuf)
        code, _ = ctx.get_status()
        assert code == 0, code
        counts = np.bincount(idx, minlength=T)
        flops = 2 * dsn.dsn_executed_macs(counts.tolist(), R, k_in, k_out, K)
        gemm_row(cfgname, lname, rname, B, us, flops, gemm_algorithmic_bytes(counts, R, k_in, k_out, K),
                 mma_floor_util(counts, R, k_in, k_out, K))
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
        us = timer.time_us(lambda i: dsn.dsn_gate(ctx, g, xs[i % nbuf], idx, None, ws), nbuf)
        add({"config": cfgname, "layer": "gate (pool + FC-ReLU-FC + arg-max)", "routing": "-", "us": round(us, 1),
             "bound": f"HBM {HBM:.0f} GB/s", "pct_of_bound": round(100 * per / us / 1e3 / HBM), "gbs": round(per / us / 1e3),
             "samples_per_s": round(B / us * 1e6)})
        us = timer.time_us(lambda i: dsn.dsn_route(ctx, idx, B, T, r), 8)
        add({"config": cfgname, "layer": "route", "routing": "-", "us": round(us, 1), "bound": "launch latency",
             "samples_per_s": round(B / us * 1e6)})

    def attention(cfgname, B, N, H, heads, idx, rname):
        if not want(cfgname, "attention core", rname):
            return
        B = B // div
        idx = idx[:B]
        r = routed(B, len(heads), idx)
        per = B * N * 4 * H * 64 * 2
        nbuf = max(2, int(2.2 * L2_BYTES // per) + 1)
        qs = [torch.randn(B, N, 3 * H * 64, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        os_ = [torch.zeros(B, N, H * 64, device=dev, dtype=torch.bfloat16) for _ in range(nbuf)]
        d = dsn.make_attention_desc(N, H, 64, heads, order=dsn.GROUPED)
        us = timer.time_us(lambda i: dsn.dsn_sliced_attention(ctx, d, r, qs[i % nbuf], os_[i % nbuf]), nbuf)
        assert ctx.get_status()[0] == 0
        hsum = sum(heads[t] for t in idx)
        gemm_row(cfgname, f"attention core (N={N})", rname, B, us, 4.0 * N * N * 64 * hsum, 2.0 * N * 4 * 64 * hsum)

    # configs 2 / 4: bottlenecks
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
    attention("cfg3", 256, 197, 6, [p_[1] for p_ in wl.vit_small_paths()], wl.idx_quota_uniform(wl.rng(3, 9), 256, 48), "uniform")
    attention("cfg5", 1024, 197, 12, [p_[1] for p_ in wl.vit_base_paths()], wl.idx_quota_uniform(wl.rng(5, 9), 1024, 8), "uniform")
    # config 5: ViT-B width
    B, paths = 1024, wl.vit_base_paths()
    gate_route("cfg5", B, 197, 768, 8)
    cases = [("all on path 7", wl.idx_all_one(B, 7)), ("all on path 0", wl.idx_all_one(B, 0)),
             ("uniform", wl.idx_quota_uniform(wl.rng(5, 9), B, 8)), ("zipf(1.2)", wl.idx_zipf(wl.rng(5, 9), B, 8))]
    for rname, idx in cases:
        for lname, Cin, Cout, act in (("qkv", 768, 2304, 0), ("proj", 768, 768, 0), ("fc1", 768, 3072, 2), ("fc2", 3072, 768, 0)):
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
    if want("cfg1", "fp32 linear", "iid"):
        c1 = wl.config1()
        x, W = torch.from_numpy(c1["x"]).to(dev), torch.from_numpy(c1["W"]).to(dev)
        y = torch.zeros(64, 1, 256, device=dev)
        r = routed(64, 4, c1["idx"])
        d = dsn.make_linear_desc(dsn.F32, 1, 256, 256, c1["k_in"], c1["k_out"], W)
        us = timer.time_us(lambda i: dsn.dsn_sliced_linear(ctx, d, r, x, y), 8)
        fl = 2 * dsn.dsn_executed_macs(np.bincount(c1["idx"], minlength=4).tolist(), 1, c1["k_in"], c1["k_out"], 1)
        add({"config": "cfg1", "layer": "fp32 linear 256x256, B=64", "routing": "iid", "us": round(us, 1),
             "tflops": round(fl / us / 1e6, 3), "bound": "launch latency", "samples_per_s": round(64 / us * 1e6)})
    return rows


TABLE_HEADER = ("| config | layer | routing | us | executed TFLOP/s | % measured BF16 peak | bound (TFLOP/s) | % of bound | GB/s | samples/s |\n"
                "|---|---|---|---|---|---|---|---|---|---|")


def row_markdown(r):
    g = lambda k: r.get(k, "-")
    bound = r.get("bound_tflops", r.get("bound", "-"))
    return (f"| {g('config')} | {g('layer')} | {g('routing')} | {g('us')} | {g('tflops')} | {g('pct_bf16_peak')} | {bound} | "
            f"{g('pct_of_bound')} | {g('gbs')} | {g('samples_per_s')} |")


# --------------------------------------------------------------------------------------------- main arm
def spawn_ranks(args):
    """`--gpus N` without a launcher: start N ranks (one process per GPU) and pass their output through."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    argv = [a for a in sys.argv[1:]]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + argv
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "WARN")
    raise SystemExit(subprocess.call(cmd, env=env))


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="dsn", choices=["dsn", "reference"])
    ap.add_argument("--workload", default="cfg5", help="one of " + ", ".join(WORKLOADS))
    ap.add_argument("--routing", default=None, help="cfg3/cfg5: uniform (default), zipf, one0, one7, gate; cfg2: gate (default) or uniform")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="leave the per-layer rows of every configuration out of the JSON line")
    ap.add_argument("--table", action="store_true", help="print the per-layer rows of every configuration as a markdown table and exit")
    ap.add_argument("--no-graph", action="store_true", help="time direct API calls instead of a CUDA-graph replay (for profilers)")
    ap.add_argument("--table-filter", default=None, help="per-layer rows: only those whose 'config layer routing' text matches this regular expression")
    ap.add_argument("--table-batch-div", type=int, default=1, help="per-layer rows: divide every batch size by this (small cases for profilers)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return
    world_env = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world_env == 1:
        spawn_ranks(args)
    if world_env > 1 and world_env != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={world_env}")

    import torch
    from paper_2109_10060_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = world_env
    if not torch.cuda.is_available() or torch.cuda.device_count() <= local_rank:
        raise SystemExit(f"rank {rank}: no CUDA device {local_rank} (the benchmark has no CPU path)")
    dist = None
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
    timer = GraphTimer(torch, use_graph=not args.no_graph)

    if args.table:
        print(TABLE_HEADER)
        collect_rows(dsn, torch, ctx, dev, peaks, timer, args.table_filter, args.table_batch_div,
                     emit=lambda r: print(row_markdown(r), flush=True))
        return

    wlk = make_workload(args.workload, dsn, torch, dev, args.batch, args.routing)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def status_ok():
        code, detail = ctx.get_status()
        if code != 0:
            raise SystemExit(f"device status {code} ({dsn.dsn_strerror(code)}) detail {detail}")

    launches0 = ctx.stats()["launches"]
    wlk.step(ctx, 0)
    launches_per_step = ctx.stats()["launches"] - launches0   # counted by the library itself, one direct step
    t_host0 = time.perf_counter()
    for i in range(args.warmup):
        wlk.step(ctx, i)
    host_us_per_step = (time.perf_counter() - t_host0) / args.warmup * 1e6   # enqueue time of the API calls (first call included)
    barrier()
    status_ok()
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
        """n steps, n a multiple of the buffer-set count when graphed."""
        if graphed:
            for _ in range(n // wlk.copies):
                graph.replay()
        else:
            for i in range(n):
                wlk.step(ctx, i)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    run_steps(2 * wlk.copies)
    e1.record(stream)
    torch.cuda.synchronize()
    est_ms = max(e0.elapsed_time(e1) / (2 * wlk.copies), 1e-4)
    # EXACTLY --steps steps are asked for; the timed region is stretched to MIN_TIMED_SECONDS where that
    # many steps would be shorter (and to a whole number of graph replays); ms_per_step = region / timed_steps
    timed_steps = max(args.steps, int(math.ceil(MIN_TIMED_SECONDS * 1e3 / est_ms)))
    timed_steps = -(-timed_steps // wlk.copies) * wlk.copies
    if world > 1:
        tmax = torch.tensor([timed_steps], dtype=torch.int64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        timed_steps = int(tmax.item())
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    e0.record(stream)
    run_steps(timed_steps)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    status_ok()

    # the same steps as direct API calls (no graph): device time per step and host time to enqueue one
    direct_n = max(wlk.copies, min(timed_steps, 50))
    torch.cuda.synchronize()
    t_host0 = time.perf_counter()
    e0.record(stream)
    for i in range(direct_n):
        wlk.step(ctx, i)
    e1.record(stream)
    host_enqueue_us = (time.perf_counter() - t_host0) / direct_n * 1e6
    torch.cuda.synchronize()
    direct_ms = e0.elapsed_time(e1) / direct_n

    # per-kernel durations: each step of the path (same kernels, one C call each) captured as its own
    # graph over the rotating buffers and replayed back to back
    parts = wlk.parts(counts)
    for _, call, _, _, _ in parts:          # consistent routing arrays and intermediates for every part
        call(ctx, 0)
    torch.cuda.synchronize()
    part_us = {}
    for pname, call, _, _, _ in parts:
        part_us[pname] = timer.time_us(lambda i, c=call: c(ctx, i % wlk.copies), wlk.copies, min_seconds=0.1)
    status_ok()

    # end to end: batch starts and ends in pinned host memory; upload, compute and download overlap
    hx, hy = wlk.e2e_io()
    streams = (torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream())
    events = [tuple(torch.cuda.Event() for _ in range(3)) for _ in range(wlk.copies)]
    for evs in events:
        evs[2].record(stream)
    torch.cuda.synchronize()
    wlk.e2e_pipeline(ctx, hx, hy, 2 * wlk.copies, streams, events)
    barrier()
    e2e_steps = max(2 * wlk.copies, min(args.steps, 40))
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
    status_ok()

    from paper_2109_10060_b200.sharding import max_over_ranks
    t = max_over_ranks(torch.tensor([ms_total], dtype=torch.float64, device=dev), dist)
    t2 = max_over_ranks(torch.tensor([ms_e2e], dtype=torch.float64, device=dev), dist)
    ms_step = float(t.item()) / timed_steps
    ms_e2e = float(t2.item())
    flops = wlk.exec_flops(counts)
    value = world * flops / (ms_step * 1e-3) / 1e12
    e2e_value = world * flops / (ms_e2e * 1e-3) / 1e12
    if rank != 0:
        return

    # roofline of the dominant grouped-GEMM launch
    info = {p[0]: p for p in parts}
    gemm_parts = [p for p in parts if p[4] in ("gemm", "chain")]
    chain = [p for p in gemm_parts if p[4] == "chain"]
    # the launch with the most executed FLOPs (the first of equals: fc1 before fc2), so that the line always describes
    # the same launch; by duration the two MLP layers of the ViT block swap places from run to run
    dom = chain[0] if chain else max((p for p in gemm_parts), key=lambda p: p[2])
    dname, dcall, dflops, dbytes, dkind = dom
    dus = part_us[dname]
    dus_burst = burst_time_us(torch, lambda i: dcall(ctx, i % wlk.copies), wlk.copies)
    ai = dflops / dbytes
    ridge = peaks["bf16_tflops"] * 1e3 / peaks["hbm_gbs"]
    sustained_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    if ai >= ridge:
        # back to back for 0.1 s the launch runs under the power cap, like the sustained cuBLAS figure: that pair is
        # the roofline fraction; the launch alone after an idle pause against the burst figure is given beside it
        ach, peak, unit, bound = dflops / dus / 1e6, sustained_peak, "TFLOP/s", "tensor"
        src = peaks["source"] + " cuBLAS bf16 matmul, sustained (launch replayed back to back for 0.1 s)"
    else:
        ach, peak, unit, bound = dbytes / dus / 1e3, peaks["hbm_gbs"], "GB/s", "hbm"
        src = peaks["source"] + " copy bandwidth"
    kernel = ("gemm_bf16_chain_kernel" if dkind == "chain" else
              ("gemm_bf16_halo_kernel" if dname.endswith("3x3") and wlk.R > 200 and max(wlk.widths) <= 128 else "gemm_bf16_pair_kernel"))
    traffic_key = f"{args.workload}:{dname.split(':')[-1]}" + (f":{args.routing}" if args.routing else "")
    roofline = {"bound": bound, "kernel": kernel, "launch": dname, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                "peak_source": src, "traffic": recorded_traffic(kernel, traffic_key),
                "algorithmic_bytes_per_launch": dbytes, "flops_per_launch": dflops, "us_per_launch": round(dus, 2),
                "arithmetic_intensity": round(ai, 1), "ridge": round(ridge, 1),
                "executed_tflops": dflops / dus / 1e6,
                "frac_of_bf16_peak_sustained": dflops / dus / 1e6 / sustained_peak,
                "alone": {"us_per_launch": round(dus_burst, 2), "executed_tflops": dflops / dus_burst / 1e6,
                          "frac_of_bf16_peak_burst": dflops / dus_burst / 1e6 / peaks["bf16_tflops"],
                          "gbs": dbytes / dus_burst / 1e3,
                          "how": "best of 8 single launches after an idle pause, the way the burst peak was taken"},
                "timing": ("one API call (route + chained launch) per replay; the route kernel's share is inside the figure"
                           if dkind == "chain" else "the launch alone in a CUDA graph of its own, replayed for 0.1 s")}
    gsel = [p for p in gemm_parts if p[4] == "gemm"]
    g_fl, g_us = sum(p[2] for p in gsel), sum(part_us[p[0]] for p in gsel)
    gemm_layers = {"layers": [p[0] for p in gsel], "executed_tflops": g_fl / g_us / 1e6, "us": round(g_us, 1),
                   "frac_of_bf16_peak_burst": g_fl / g_us / 1e6 / peaks["bf16_tflops"],
                   "frac_of_bf16_peak_sustained": g_fl / g_us / 1e6 / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                   "per_layer": {p[0]: {"us": round(part_us[p[0]], 1), "tflops": round(p[2] / part_us[p[0]] / 1e6, 1),
                                        "frac_of_bf16_peak_burst": round(p[2] / part_us[p[0]] / 1e6 / peaks["bf16_tflops"], 3)}
                                 for p in gsel}}

    out = {
        "metric": "sliced_gemm_executed_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "timed_steps": timed_steps, "warmup": args.warmup, "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_title(args.workload), "name": wlk.name, "batch_per_gpu": wlk.B,
                   "routing": wlk.routing_name, "path": wlk.path, "flops": wlk.flops_note,
                   "l2": f"inputs and outputs rotate over {wlk.copies} buffer sets; one set's input is "
                         f"{wlk.x_host_bits.nbytes / 1e6:.0f} MB (L2 126 MB)",
                   "launch": "CUDA graph replay of the public-API step" if graphed else "direct calls",
                   "timed_region": f"{timed_steps} steps = max(--steps, {MIN_TIMED_SECONDS} s worth), {ms_total:.1f} ms",
                   "routing_histogram": counts.tolist(), "parallelism": f"batch shards x{world}, no collective"},
        "samples_per_s": world * wlk.B / (ms_step * 1e-3),
        "pct_bf16_peak_burst": 100 * value / world / peaks["bf16_tflops"],
        "pct_bf16_peak_sustained": 100 * value / world / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
        "pct_bf16_peak_nominal": 100 * value / world / NOMINAL_BF16_TFLOPS,
        "direct_calls": {"ms_per_step": direct_ms, "host_enqueue_us_per_step": round(host_enqueue_us, 1),
                         "host_enqueue_us_per_step_first_calls": round(host_us_per_step, 1),
                         "note": "the same steps issued as plain API calls without a graph"},
        "kernel_us": {k: round(v, 2) for k, v in part_us.items()},
        "roofline": roofline,
        "gemm_layers": gemm_layers,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": int(hx.numel() * 2),
                "d2h_bytes_per_step": int(hy.numel() * 2), "ms_per_step": ms_e2e,
                "how": "the public-API step per batch; upload, compute and download pipelined on three streams"},
        "gpu_launches": launches_per_step * timed_steps,
        "gpu_launches_per_step": launches_per_step,
        "library_stats": ctx.stats(),
        "clocks": clocks,
    }
    if not args.no_cpu_baseline and world == 1:
        n = {"cfg5": 8, "cfg3": 16}.get(args.workload, min(wlk.B, 128))
        samples = wlk.oracle_samples(n)
        t0 = time.perf_counter()
        f_cpu = wlk.oracle_run(samples)
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": f_cpu / dt / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
                               "sample": f"{n} of {wlk.B} samples; {wlk.oracle_what}; {dt:.1f} s wall"}
    if not args.no_per_config and world == 1:
        del wlk
        torch.cuda.empty_cache()
        out["per_config"] = collect_rows(dsn, torch, ctx, dev, peaks, timer, args.table_filter, args.table_batch_div)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
