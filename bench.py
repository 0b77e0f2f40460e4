#!/usr/bin/env python
"""Benchmark of the variance-based gradient compression hot path on B200.

One "step" is one pass of the whole hot path over one mini-batch of synthetic input:
squared per-example gradient sums for every layer (vgc_sqgrad_conv / vgc_sqgrad_linear) into
the flat buffer s, one compressor step over the flat buffer (vgc_compress), and the decode of
W packed messages into the dense update (vgc_decode_accumulate).

Default workload: the ResNet-50-shaped flat buffer (53 conv + 1 fc weight tensors, 25.5 M
weights, batch 32, 224x224 input) -- the paper's ImageNet workload shape and the only
configuration that exercises all three parts at a size that is not cache resident.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload resnet50|mlp|dense|vgg16]
    python bench.py --impl reference ...      # times the CPU oracle on a bounded sample

Prints ONE JSON line on rank 0.  Besides the timed steps the default single-GPU run also (outside the timed
region) checks one step against the CPU oracle ("parity"), measures the TF32 matmul peak the tensor roofline
is quoted against, times the sqgrad pass over >= 2 s with the clock sampler running, and times the two
configurations that have no sqgrad part: the VGG-16-sized compress ("config4") and the decode sweep ("config5").
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

import numpy as np
import torch

METRIC = "hot-path throughput (sqgrad + compress + decode), parameters per second"
UNIT = "Gparam/s"

WORKLOADS = {
    # name: (config id, layer table, batch, x kind, delta std, W messages, alpha)
    "dense": (0, "dense_layers", 32, "normal", 1e-2, 4, 2.0),
    "mlp": (1, "mlp_layers", 128, "relu_normal", 1e-3, 8, 2.0),
    "resnet50": (2, "resnet50_layers", 32, "half_normal", 1e-4, 8, 2.0),
    "vgg16": (3, "vgg16_layers", 64, "half_normal", 1e-4, 0, 2.0),      # compress only
    # a flat buffer of --n-params weights in 16 equal tensors: compress + decode only (small profiling case)
    "flat": (4, None, 64, "half_normal", 1e-4, 4, 2.0),
}
ZETA = 0.999


HBM_NOMINAL_GBS = 8000.0       # the "about 8 TB/s" the target is also quoted against


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def ncu_traffic():
    """DRAM traffic figures read off ncu captures (profiles/ncu_traffic.json names the captures and the library
    version they were taken on); None where the file has no figure."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    return json.load(open(path)) if os.path.exists(path) else {}


def measure_tf32_peak(sustain_s: float = 2.0):
    """TF32 tensor-core peak of this GPU measured like the bf16 figures of MEASURED_PEAKS.json: torch.matmul
    (cuBLAS, TF32 allowed) on 8192^3, best of 10 single calls (burst) and back to back for `sustain_s` seconds
    (sustained, under the power cap).  Returns (burst TFLOP/s, sustained TFLOP/s)."""
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        n = 8192
        a = torch.randn(n, n, device="cuda"); b = torch.randn(n, n, device="cuda"); c = torch.empty(n, n, device="cuda")
        flops = 2.0 * n ** 3
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(a, b, out=c); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
            time.sleep(0.02)                                   # let the clocks recover between single calls
        reps = max(int(sustain_s / (best * 1e-3)), 10)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize()
        sustained = flops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12
        return flops / (best * 1e-3) / 1e12, sustained
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev


# ----------------------------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            if len(row) < 7:
                continue
            try:
                sm.append(float(row[0])); smax.append(float(row[1]))
            except ValueError:
                continue
            for name, val in zip(names, row[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# the pipeline under test
# ----------------------------------------------------------------------------------------------
class HotPath:
    """All device buffers of one worker and the launches of one step."""

    def __init__(self, name: str, worker: int, n_input_sets: int, n_g_sets: int, device="cuda",
                 n_params: int = 1 << 25, n_streams: int = 5, algorithm: str = "basic", batch_layers: bool = True,
                 exact_conv: bool = False):
        import paper_1802_06058_b200 as vgc
        from paper_1802_06058_b200 import workloads
        self.vgc, self.wl = vgc, workloads
        cfg, table, self.batch, x_kind, delta_std, self.W, self.alpha = WORKLOADS[name]
        self.name, self.cfg = name, cfg
        if table is None:
            self.layers = []
            self.offsets = np.linspace(0, n_params, 17).astype(np.uint32)
        else:
            self.layers = getattr(workloads, table)()
            self.offsets = workloads.group_offsets(self.layers)
        self.n = int(self.offsets[-1])
        self.K = len(self.offsets) - 1
        self.offs_dev = vgc.offsets_tensor(self.offsets)
        self.compress_only = name in ("vgg16", "flat")
        self.fused = False
        self.hybrid = algorithm == "hybrid"                # Algorithm 2 instead of Algorithm 1
        self.exact_conv = exact_conv                       # per-example conv statistic (cross terms kept)
        self.tau = 0.0
        dev = device
        B = self.batch
        self.scale = 1.0 / (B * B)
        f32 = dict(dtype=torch.float32, device=dev)
        self.s = torch.zeros(self.n, **f32)
        self.r = torch.zeros(self.n, **f32)
        self.v = torch.zeros(self.n, **f32)
        self.u = torch.zeros(self.n, **f32)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        if self.hybrid:
            self.out = vgc.HybridMessageBuffers(self.n, self.n, with_mask=False, device=dev)
        else:
            self.out = vgc.MessageBuffers(self.n, self.K, self.n, with_mask=False, device=dev)
        self.ws_c = torch.empty(max(vgc.vgc_compress_workspace_bytes(self.n, self.K),
                                    vgc.vgc_compress_hybrid_workspace_bytes(self.n)), dtype=torch.uint8, device=dev)
        self.flops_useful = 0
        self.flops_issued = 0.0      # in TF32-product equivalents: what the tensor pipe is asked to do
        self.inputs = []
        if self.compress_only:
            gs = [workloads.per_parameter_gs(self.n, B, delta_std, workloads.seed_for(cfg, worker, t, 0, 2), dev)
                  for t in range(n_g_sets)]
            self.g_sets = [g for g, _ in gs]
            self.s_sets = [s for _, s in gs]
            self.ws_s = None
        else:
            vgc.vgc_sqgrad_plan_hint(n_streams)
            ws_bytes = 16
            # conv layers of one geometry go to the library together (one launch per group of up to 8)
            groups = {}
            for li, spec in enumerate(self.layers):
                key = (spec.kind, spec.cin, spec.cout, spec.k, spec.stride, spec.pad, spec.hin) if batch_layers and spec.kind == "conv" else li
                groups.setdefault(key, []).append(li)
            self.groups = [g[i:i + 8] for g in groups.values() for i in range(0, len(g), 8)]
            # long groups first: the short ones fill the gaps at the end of the pass
            self.groups.sort(key=lambda g: -sum(2 * np.prod(self.layers[li].gemm_mnk(B)) for li in g))
            for li, spec in enumerate(self.layers):
                M, N, K = spec.gemm_mnk(B)
                self.flops_useful += 2 * M * N * K
                # fp32 accuracy costs three TF32 products per algorithmic one; the TMA-fed form (all 1x1 convs) takes
                # its two cross terms in bf16, at half the TF32 cost each
                bf16_cross = spec.kind == "conv" and spec.k == 1 and not exact_conv
                self.flops_issued += 2 * M * N * K * (2.0 if bf16_cross else 3.0)
            for g in self.groups:
                spec = self.layers[g[0]]
                if spec.kind == "conv":
                    geo = (B, spec.cin, spec.hin, spec.hin, spec.cout, spec.k, spec.k, spec.stride, spec.stride,
                           spec.pad, spec.pad)
                    ws_bytes = max(ws_bytes, vgc.vgc_sqgrad_conv_batch_workspace_bytes(len(g), *geo, exact=exact_conv),
                                   vgc.vgc_sqgrad_conv_workspace_bytes(*geo))      # the end-to-end leg calls layer by layer
                else:
                    ws_bytes = max(ws_bytes, vgc.vgc_sqgrad_linear_workspace_bytes(B, spec.cin, spec.cout))
            self.ws_s = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
            # independent layers are spread over a few streams (each with its own workspace) so that one
            # layer's tail and the next one's start overlap; the whole step is then replayed as a CUDA graph
            self.n_streams = n_streams
            self.side = [torch.cuda.Stream() for _ in range(max(n_streams - 1, 0))]
            self.ws_side = [torch.zeros(ws_bytes, dtype=torch.uint8, device=dev) for _ in self.side]
            for t in range(n_input_sets):
                self.inputs.append([workloads.layer_inputs(spec, B, cfg, worker, t, li, x_kind, delta_std, dev)
                                    for li, spec in enumerate(self.layers)])
            # g is an input of the compressor made by the harness: one noise draw per step whose
            # variance matches the squared-gradient sums (g_t = z_t * sqrt(s)), like a mini-batch
            # gradient under pure noise
            self.sqgrad(0)
            root_s = self.s.sqrt()
            gen = torch.Generator(device=dev); gen.manual_seed(workloads.seed_for(cfg, worker, 0, 0, 3))
            self.g_sets = [torch.empty(self.n, **f32).normal_(generator=gen).mul_(root_s) for _ in range(n_g_sets)]
            self.s_sets = None
        # messages of the other W-1 workers: generated inputs (their own noise draws, compressed once)
        self.others = []
        if self.hybrid:
            # the fixed threshold of the hybrid: the median noise scale of the buffer, so that about half
            # of the parameters can reach it at all
            self.tau = float((self.s if self.s_sets is None else self.s_sets[0]).sqrt().median().item())
        if self.W > 1:
            root_s = (self.s if self.s_sets is None else self.s_sets[0]).sqrt()
            rr = torch.zeros(self.n, **f32); vv = torch.zeros(self.n, **f32)
            for w in range(1, self.W):
                gen = torch.Generator(device=dev); gen.manual_seed(workloads.seed_for(cfg, worker + w, 0, 0, 3))
                gw = torch.empty(self.n, **f32).normal_(generator=gen).mul_(root_s)
                rr.zero_(); vv.zero_()
                if self.hybrid:
                    mb = vgc.HybridMessageBuffers(self.n, self.n, device=dev)
                    vgc.vgc_compress_hybrid(gw, self.s if self.s_sets is None else self.s_sets[0], rr, vv,
                                            self.alpha, ZETA, self.tau, mb, self.ws_c)
                else:
                    mb = vgc.MessageBuffers(self.n, self.K, self.n, device=dev)
                    vgc.vgc_compress(gw, self.s if self.s_sets is None else self.s_sets[0], rr, vv, self.offs_dev,
                                     self.alpha, ZETA, mb, self.ws_c)
                torch.cuda.synchronize()
                nnz = int(mb.counters[0].item())
                mb.words = mb.words[:max(nnz, 4)].clone()          # keep only what was written
                self.others.append(mb)
            del rr, vv

    # -- launches -------------------------------------------------------------------------------
    def sqgrad(self, t: int, into_v: bool = False):
        """Squared-gradient sums of every layer into s (or, fused form, added straight into v)."""
        vgc = self.vgc
        if self.compress_only:
            return
        target = self.v if into_v else self.s
        ins = self.inputs[t % len(self.inputs)]
        main = torch.cuda.current_stream()
        for st in self.side:
            st.wait_stream(main)
        for gi, g in enumerate(self.groups):
            spec = self.layers[g[0]]
            Ss = [target[int(self.offsets[li]):int(self.offsets[li + 1])] for li in g]
            lane = gi % self.n_streams
            stream = main if lane == 0 else self.side[lane - 1]
            ws = self.ws_s if lane == 0 else self.ws_side[lane - 1]
            if spec.kind == "conv":
                vgc.vgc_sqgrad_conv_batch([ins[li][0] for li in g], [ins[li][1] for li in g], (spec.k, spec.k),
                                          (spec.stride, spec.stride), (spec.pad, spec.pad), self.scale, Ss,
                                          accumulate=into_v, ws=ws, stream=stream, exact=self.exact_conv)
            else:
                vgc.vgc_sqgrad_linear(ins[g[0]][0], ins[g[0]][1], self.scale, Ss[0], accumulate=into_v, ws=ws,
                                      stream=stream)
        for st in self.side:
            main.wait_stream(st)

    def per_layer_times(self, reps: int = 5):
        """Median device time of each sqgrad library call (a layer, or a group of same-shaped layers) in ms."""
        vgc = self.vgc
        out = []
        ins = self.inputs[0]
        for g in self.groups:
            spec = self.layers[g[0]]
            Ss = [self.s[int(self.offsets[li]):int(self.offsets[li + 1])] for li in g]
            def call():
                if spec.kind == "conv":
                    vgc.vgc_sqgrad_conv_batch([ins[li][0] for li in g], [ins[li][1] for li in g], (spec.k, spec.k),
                                              (spec.stride, spec.stride), (spec.pad, spec.pad), self.scale, Ss,
                                              ws=self.ws_s)
                else:
                    vgc.vgc_sqgrad_linear(ins[g[0]][0], ins[g[0]][1], self.scale, Ss[0], ws=self.ws_s)
            call(); torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for _ in range(10):
                    call()
            times = []
            for r in range(reps + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                graph.replay()
                e1.record()
                torch.cuda.synchronize()
                if r >= 2:
                    times.append(e0.elapsed_time(e1) / 10)
            M, N, K = spec.gemm_mnk(self.batch)
            ms = statistics.median(times)
            out.append({"layer": "+".join(self.layers[li].name for li in g), "layers": len(g), "M": M, "N": N, "K": K,
                        "ms": round(ms, 4),
                        "useful_tflops": round(len(g) * 2 * M * N * K / (ms * 1e-3) / 1e12, 2)})
        return out

    def compress(self, t: int, fused: bool = False):
        s = None if fused else (self.s if self.s_sets is None else self.s_sets[t % len(self.s_sets)])
        if self.hybrid:
            self.vgc.vgc_compress_hybrid(self.g_sets[t % len(self.g_sets)], s, self.r, self.v, self.alpha, ZETA,
                                         self.tau, self.out, self.ws_c)
            return
        self.vgc.vgc_compress(self.g_sets[t % len(self.g_sets)], s, self.r, self.v, self.offs_dev, self.alpha,
                              ZETA, self.out, self.ws_c)

    def decode(self, t: int):
        if self.W == 0:
            return
        # u = mean of the W messages, every element written (no clearing pass, u is not read)
        if self.hybrid:
            self.vgc.vgc_decode_sum_hybrid([self.out] + self.others, self.tau, 1.0 / self.W, self.u, self.status)
            return
        self.vgc.vgc_decode_sum([self.out] + self.others, self.offs_dev, 1.0 / self.W, self.u, self.status)

    def step(self, t: int, marks=None):
        fused = self.fused and not self.compress_only
        self.sqgrad(t, into_v=fused)
        if marks: marks[0].record()
        self.compress(t, fused=fused)
        if marks: marks[1].record()
        self.decode(t)
        if marks: marks[2].record()


class GraphedStep:
    """The launches of one step captured once per input set and replayed (CUDA graph): the step is a
    fixed sequence of ~60 small launches, so replaying removes the host launch cost from the loop."""

    def __init__(self, hp: HotPath, n_variants: int):
        self.graphs = []
        self.launches = []
        for t in range(n_variants):
            hp.step(t)                                   # eager once: first-call set-up happens outside capture
        torch.cuda.synchronize()
        for t in range(n_variants):
            before = hp.vgc.vgc_kernel_launch_count()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                hp.step(t)
            self.launches.append(hp.vgc.vgc_kernel_launch_count() - before)
            self.graphs.append(g)
        self.hp = hp

    def replay(self, t: int):
        self.graphs[t % len(self.graphs)].replay()


def run_device_timed(hp: HotPath, steps: int, warmup: int, dist_on: bool, use_graph: bool = True):
    vgc = hp.vgc
    ev = lambda: torch.cuda.Event(enable_timing=True)
    if use_graph:
        return run_graph_timed(hp, steps, warmup, dist_on)
    for t in range(warmup):
        hp.step(t)
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    marks = [[ev() for _ in range(4)] for _ in range(steps)]
    launches0 = vgc.vgc_kernel_launch_count()
    start, stop = ev(), ev()
    start.record()
    for i in range(steps):
        marks[i][3].record()
        hp.step(warmup + i, marks[i])
    stop.record()
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    launches = vgc.vgc_kernel_launch_count() - launches0
    total_ms = start.elapsed_time(stop)
    sq = [m[3].elapsed_time(m[0]) for m in marks]
    co = [m[0].elapsed_time(m[1]) for m in marks]
    de = [m[1].elapsed_time(m[2]) for m in marks]
    return total_ms, sq, co, de, launches


def run_graph_timed(hp: HotPath, steps: int, warmup: int, dist_on: bool):
    """Timed region = K graph replays (whole steps) bracketed by events; the per-section split comes from
    a second, untimed pass in which each section is replayed as its own graph."""
    ev = lambda: torch.cuda.Event(enable_timing=True)
    n_var = len(hp.g_sets)
    gs = GraphedStep(hp, n_var)
    for t in range(warmup):
        gs.replay(t)
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    start, stop = ev(), ev()
    start.record()
    for i in range(steps):
        gs.replay(warmup + i)
    stop.record()
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    total_ms = start.elapsed_time(stop)
    launches = sum(gs.launches[(warmup + i) % n_var] for i in range(steps))
    # section split (outside the timed region): each section replayed as its own graph, rotating over the
    # same per-step inputs as the timed steps so that the compressor state keeps evolving the same way
    secs = []
    for fn in (hp.sqgrad, hp.compress, hp.decode):
        graphs = []
        for t in range(n_var):
            fn(t)
        torch.cuda.synchronize()
        for t in range(n_var):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn(t)
            graphs.append(g)
        times = []
        for r in range(max(steps, 5) + 2):
            e0, e1 = ev(), ev()
            e0.record(); graphs[r % n_var].replay(); e1.record()
            torch.cuda.synchronize()
            if r >= 2:
                times.append(e0.elapsed_time(e1))
        secs.append(times)
    return total_ms, secs[0], secs[1], secs[2], launches


def sustained_sqgrad(hp: HotPath, device_index: int, seconds: float = 2.0):
    """The sqgrad pass replayed back to back for about `seconds` with the clock sampler running: (ms per pass, clocks)."""
    n_var = len(hp.inputs)
    graphs = []
    for t in range(n_var):
        hp.sqgrad(t)
    torch.cuda.synchronize()
    for t in range(n_var):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            hp.sqgrad(t)
        graphs.append(g)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(20):
        graphs[i % n_var].replay()
    e1.record()
    torch.cuda.synchronize()
    reps = max(int(seconds / (e0.elapsed_time(e1) / 20 * 1e-3)), 20)
    sampler = ClockSampler(device_index)
    sampler.start()
    e0.record()
    for i in range(reps):
        graphs[i % n_var].replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    return e0.elapsed_time(e1) / reps, clocks


def run_e2e(hp: HotPath, steps: int, warmup: int):
    """Same step end to end from HOST buffers: every step copies its inputs (each layer's x and delta, and g)
    from pinned host memory to the device, runs the path, and reads the message (counters, then the packed
    words) back to the host.  Layered workloads go through the C ABI's vgc_step_host, which does the copies
    itself; the compress-only workloads copy g and s with torch and call vgc_compress."""
    vgc = hp.vgc
    words_host = torch.empty(hp.n, dtype=torch.int32).pin_memory()
    counters_host = torch.zeros(4, dtype=torch.int32).pin_memory()
    d2h_total = 0
    if hp.compress_only:
        g_host, s_host = hp.g_sets[0].cpu().pin_memory(), hp.s_sets[0].cpu().pin_memory()
        h2d = 8 * hp.n

        def one(t):
            nonlocal d2h_total
            hp.g_sets[0].copy_(g_host, non_blocking=True)
            hp.s_sets[0].copy_(s_host, non_blocking=True)
            hp.compress(0); hp.decode(0)
            counters_host.copy_(hp.out.counters, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            nnz = min(int(counters_host[0]), hp.n)
            words_host[:nnz].copy_(hp.out.words[:nnz], non_blocking=True)
            torch.cuda.current_stream().synchronize()
            d2h_total += 16 + 4 * nnz
    else:
        layers = []
        h2d = 4 * hp.n
        for spec, (x, d) in zip(hp.layers, hp.inputs[0]):
            xh, dh = x.cpu().pin_memory(), d.cpu().pin_memory()
            h2d += 4 * (xh.numel() + dh.numel())
            layers.append({"is_conv": spec.kind == "conv", "B": hp.batch, "C": spec.cin, "H": spec.hin, "W": spec.hin,
                           "Cout": spec.cout, "Kh": spec.k, "Kw": spec.k, "stride": spec.stride, "pad": spec.pad,
                           "x_host": xh, "delta_host": dh, "x_dev": x, "delta_dev": d})
        g_host = hp.g_sets[0].cpu().pin_memory()

        def one(t):
            nonlocal d2h_total
            nnz, _, _, _ = vgc.vgc_step_host(layers, g_host, hp.g_sets[0], hp.s, hp.r, hp.v, hp.offs_dev, hp.alpha,
                                             ZETA, hp.scale, hp.out, words_host, counters_host, hp.ws_s, hp.ws_c)
            hp.decode(0)
            torch.cuda.current_stream().synchronize()
            d2h_total += 16 + 4 * min(nnz, hp.n)

    for t in range(warmup):
        one(t)
    torch.cuda.synchronize()
    d2h_total = 0
    t0 = time.perf_counter()
    for t in range(steps):
        one(t)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    return dt * 1e3 / steps, h2d, d2h_total // max(steps, 1)


# ----------------------------------------------------------------------------------------------
# parity of what was timed (outside the timed region)
# ----------------------------------------------------------------------------------------------
def sample_entries(spec, rng, at_least: int):
    """Flat weight indices of one layer to compare with the oracle: one in every 128 x 128 tile of its
    [Cout] x [C*k*k] result (the kernels' tile grid), the four corners, and random ones up to `at_least`
    (every entry of a layer that has fewer)."""
    M, N = spec.cout, spec.cin * spec.k * spec.k
    if M * N <= at_least:
        return np.arange(M * N)
    rows0, cols0 = np.arange(0, M, 128), np.arange(0, N, 128)
    rr = np.minimum(rows0[:, None] + rng.integers(0, 128, (rows0.size, cols0.size)), M - 1)
    cc = np.minimum(cols0[None, :] + rng.integers(0, 128, (rows0.size, cols0.size)), N - 1)
    per_tile = (rr * N + cc).reshape(-1)
    corners = np.array([0, N - 1, (M - 1) * N, M * N - 1])
    extra = rng.integers(0, M * N, max(at_least - per_tile.size, 0))
    return np.unique(np.concatenate([per_tile, corners, extra]))


def sqgrad_sampled_error(hp: "HotPath", t: int, at_least: int, seed: int = 0) -> float:
    """Largest relative error of hp.s (as left by hp.sqgrad(t)) against the oracle over sampled entries of every layer."""
    import oracle
    rng = np.random.default_rng(seed)
    worst = 0.0
    ins = hp.inputs[t % len(hp.inputs)]
    for li, spec in enumerate(hp.layers):
        x, d = ins[li]
        idx = sample_entries(spec, rng, at_least)
        got = hp.s[int(hp.offsets[li]):int(hp.offsets[li + 1])].cpu().numpy()[idx].astype(np.float64)
        if spec.kind == "conv":
            ref = oracle.sqgrad_conv_entries(x.cpu().numpy(), d.cpu().numpy(), (spec.k, spec.k), (spec.stride, spec.stride),
                                             (spec.pad, spec.pad), hp.scale, idx)
        else:
            ref = oracle.sqgrad_linear(x.cpu().numpy(), d.cpu().numpy(), scale=hp.scale).reshape(-1)[idx]
        ref = ref.astype(np.float64)
        rel = np.abs(got - ref) / np.maximum(np.abs(ref), 1e-300)
        rel[(ref == 0) & (got == 0)] = 0.0
        worst = max(worst, float(rel.max()))
    return worst


def parity_check(hp: "HotPath", sqgrad_samples: int = 0) -> dict:
    """One more step of the pipeline as it was timed (same buffers, streams and launch configuration), compared with
    the CPU oracle fed the very same bytes: the compressor's message and state bit for bit, the decoded update within
    1e-6, and (sqgrad_samples > 0) sampled entries of the squared-gradient sums."""
    import oracle
    out = {}
    t = 0
    if sqgrad_samples and not hp.compress_only:
        hp.sqgrad(t)
        torch.cuda.synchronize()
        out["sqgrad_max_rel"] = sqgrad_sampled_error(hp, t, sqgrad_samples)
        out["sqgrad_entries_per_layer"] = f">= {sqgrad_samples} (one per 128x128 tile at least)"
    if hp.hybrid:
        return out
    g = hp.g_sets[t % len(hp.g_sets)]
    s = hp.s if hp.s_sets is None else hp.s_sets[t % len(hp.s_sets)]
    r0, v0 = hp.r.cpu().numpy().copy(), hp.v.cpu().numpy().copy()
    hp.out.counters.zero_()
    hp.compress(t)
    hp.decode(t)
    torch.cuda.synchronize()
    got = hp.out.read()
    want = oracle.compress(g.cpu().numpy(), s.cpu().numpy(), r0, v0, hp.offsets, hp.alpha, ZETA, want_mask=False)
    out["message_bit_exact"] = bool(got["dev_status"] == 0 and got["nnz"] == want.nnz and got["n_dropped"] == want.n_dropped
                                    and np.array_equal(got["words"], want.words)
                                    and np.array_equal(got["group_exp"], want.group_exp))
    out["state_bit_exact"] = bool(np.array_equal(hp.r.cpu().numpy().view(np.uint32), r0.view(np.uint32))
                                  and np.array_equal(hp.v.cpu().numpy().view(np.uint32), v0.view(np.uint32)))
    out["nnz_checked"] = int(want.nnz)
    if hp.W:
        msgs = [(want.words, want.group_exp)]
        for o in hp.others:
            k = int(o.counters[0].item())
            msgs.append((o.words[:k].cpu().numpy().view(np.uint32), o.group_exp[:o.K].cpu().numpy()))
        ref = np.zeros(hp.n, np.float32)
        oracle.decode_accumulate(msgs, hp.offsets, 1.0 / hp.W, ref)
        u = hp.u.cpu().numpy()
        out["decode_max_abs"] = float(np.abs(u.astype(np.float64) - ref).max())
        out["decode_bit_exact"] = bool(np.array_equal(u.view(np.uint32), ref.view(np.uint32)))
        out["decode_status"] = int(hp.status.item())
    return out


# ----------------------------------------------------------------------------------------------
# the configurations without a sqgrad part: VGG-16-sized compress, decode sweep
# ----------------------------------------------------------------------------------------------
def time_graph(fn, reps: int = 10, warm: int = 3) -> float:
    """Median device time in ms of fn() replayed as a CUDA graph (fn only enqueues work)."""
    fn(); torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        fn()
    times = []
    for r in range(reps + warm):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); graph.replay(); e1.record()
        torch.cuda.synchronize()
        if r >= warm:
            times.append(e0.elapsed_time(e1))
    return statistics.median(times)


def config4_compress(pk, steps: int = 8):
    """VGG-16-shaped flat buffer (138,344,128 weights in 16 tensors, batch-64 statistics per parameter): compress only."""
    hp = HotPath("vgg16", worker=0, n_input_sets=0, n_g_sets=2)
    n = hp.n
    graphs = []
    for t in range(2):
        hp.compress(t)
    torch.cuda.synchronize()
    for t in range(2):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            hp.compress(t)
        graphs.append(g)
    times = []
    for i in range(steps + 3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); graphs[i % 2].replay(); e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            times.append(e0.elapsed_time(e1))
    ms = statistics.mean(times)
    c = hp.out.read()
    nbytes = 24 * n + 8 * c["n_criterion"] + 4 * c["nnz"]
    gbs = nbytes / (ms * 1e-3) / 1e9
    res = {"workload": "vgg16 flat buffer, compress only", "n_params": n, "groups": hp.K, "alpha": hp.alpha, "ms": ms,
           "gparam_s": n / (ms * 1e-3) / 1e9, "gbs": gbs, "frac_of_measured_hbm": gbs / pk["hbm_gbs"],
           "frac_of_8tbs": gbs / HBM_NOMINAL_GBS, "send_density": c["n_criterion"] / n, "nnz": c["nnz"],
           "dev_status": c["dev_status"], "steps": steps}
    del hp
    torch.cuda.empty_cache()
    return res


def config5_decode_sweep(pk):
    """vgc_decode_accumulate over N in {ResNet-50, VGG-16 buffer} x W in {4, 16, 64} x density in {1e-4, 1e-3, 1e-2}
    generated messages (sorted distinct uniform indices, codes from the quantiser's grid; per-tensor exponents shared by
    the workers up to +-1, as workers of one job have them), plus per N one point where all W = 16 messages share one
    index set and one where every message draws its exponents independently over 13 binades (workers with nothing in
    common: the decoder's ordered form).  Bytes: 'strict' counts 4 B per word and 8 B (read + write) per element
    touched; 'moved' is what the form that ran has to move -- sparse calls (atomics) one 32-byte sector read and written
    per word plus the word, dense calls the whole of u once in and out plus the words."""
    import paper_1802_06058_b200 as vgc
    from paper_1802_06058_b200 import workloads
    rows = []
    for net in ("resnet50", "vgg16"):
        layers = getattr(workloads, net + "_layers")()
        offs = workloads.group_offsets(layers)
        n = int(offs[-1])
        offs_dev = vgc.offsets_tensor(offs)
        u = torch.zeros(n, dtype=torch.float32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        points = ([(W, rho, False, True) for W in (4, 16, 64) for rho in (1e-4, 1e-3, 1e-2)] + [(16, 1e-3, True, True)] +
                  [(16, 1e-2, False, False)])
        for W, rho, shared, common_exps in points:
            mask = None
            if shared:
                gen = torch.Generator(device="cuda"); gen.manual_seed(5)
                mask = torch.empty(n, device="cuda").uniform_(generator=gen) < rho
            msgs = [workloads.random_message(n, offs, rho, workloads.seed_for(4, w, 1 if shared else 0, 0, 2), "cuda",
                                             index_mask=mask, exp_seed=workloads.seed_for(4, 0, 0, 0, 3) if common_exps else None)
                    for w in range(W)]
            triples = [(m[0], torch.tensor([m[0].numel()], dtype=torch.int32, device="cuda"), m[1]) for m in msgs]
            sum_nnz = sum(m[0].numel() for m in msgs)
            ms = time_graph(lambda: vgc.vgc_decode_accumulate(triples, offs_dev, 1.0 / W, u, status))
            dense = sum_nnz * 8 >= n
            moved = (4 * sum_nnz + 8 * n) if dense else (4 + 64) * sum_nnz
            rows.append({"net": net, "n": n, "W": W, "density": rho, "shared_index_set": shared,
                         "exponents": "shared per tensor +-1" if common_exps else "independent per message", "sum_nnz": sum_nnz,
                         "form": "tiles in shared memory" if dense else "atomics", "ms": ms,
                         "gelem_s": sum_nnz / (ms * 1e-3) / 1e9, "gbs_strict": 12 * sum_nnz / (ms * 1e-3) / 1e9,
                         "gbs_moved": moved / (ms * 1e-3) / 1e9,
                         "moved_frac_of_measured_hbm": moved / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                         "atomics_per_s": None if dense else sum_nnz / (ms * 1e-3)})
            del msgs, triples
        assert int(status.item()) == 0
        del u
        torch.cuda.empty_cache()
    return rows


# ----------------------------------------------------------------------------------------------
# one small launch of every kernel of the library (for ncu captures; see profiles/)
# ----------------------------------------------------------------------------------------------
def profile_kernels():
    """Runs every kernel form once on a small case (after one warm-up call each): ResNet-50 layer shapes at batch 4-8
    for the squared-gradient kernels, a flat buffer of 2^24 parameters (state larger than L2) for the compressor, the
    hybrid compressor, the decoder and the index coder.  Prints one line per case; meant to run under ncu."""
    import paper_1802_06058_b200 as vgc
    from paper_1802_06058_b200 import workloads
    dev = "cuda"
    conv_cases = [  # name, layers, B, C, H, Cout, k, stride, pad
        ("1x1 both tiles by TMA, bf16 cross terms (layer-3 expansion)", 2, 8, 256, 14, 1024, 1, 1, 0),
        ("1x1 roles swapped (layer-1 reduction, Cout 64)", 2, 4, 256, 56, 64, 1, 1, 0),
        ("3x3 three taps, width % 4 == 0 (layer-1)", 1, 4, 64, 56, 64, 3, 1, 1),
        ("3x3 three taps, width % 4 == 2 (layer-3)", 2, 8, 256, 14, 256, 3, 1, 1),
        ("3x3 stride 2 three taps (layer-2 first block)", 1, 4, 128, 56, 128, 3, 2, 1),
        ("7x7 stride 2 seven taps (first layer)", 1, 4, 3, 224, 64, 7, 2, 3),
        ("1x1 on 7x7 planes: repacked channel-major (layer-4 expansion)", 2, 8, 512, 7, 2048, 1, 1, 0),
        ("1x1 stride 2: subsampled planes (layer-3 downsample)", 1, 8, 512, 28, 1024, 1, 2, 0),
        ("3x3 on 7x7 planes: padded planes + three taps (layer-4)", 1, 8, 512, 7, 512, 3, 1, 1),
        ("5x5: element-wise gather (not a ResNet shape)", 1, 4, 64, 28, 128, 5, 1, 2),
    ]
    for name, nl, B, C, H, Cout, k, st, pd in conv_cases:
        Ho = (H + 2 * pd - k) // st + 1
        xs = [torch.randn(B, C, H, H, device=dev).abs_() for _ in range(nl)]
        ds = [torch.randn(B, Cout, Ho, Ho, device=dev) * 1e-4 for _ in range(nl)]
        Ss = [torch.empty(Cout * C * k * k, device=dev) for _ in range(nl)]
        ws = torch.zeros(vgc.vgc_sqgrad_conv_batch_workspace_bytes(nl, B, C, H, H, Cout, k, k, st, st, pd, pd), dtype=torch.uint8, device=dev)
        for _ in range(2):
            vgc.vgc_sqgrad_conv_batch(xs, ds, (k, k), (st, st), (pd, pd), 1.0 / (B * B), Ss, ws=ws)
        torch.cuda.synchronize()
        print(json.dumps({"case": "sqgrad_conv: " + name, "layers": nl, "B": B, "M": Cout, "N": C * k * k, "K": B * Ho * Ho,
                          "gflop": nl * 2 * Cout * C * k * k * B * Ho * Ho / 1e9}))
    # per-example statistic (kExact), dense layers (tensor cores and CUDA cores)
    B, C, H, Cout = 8, 256, 14, 256
    x = torch.randn(B, C, H, H, device=dev); d = torch.randn(B, Cout, H, H, device=dev) * 1e-4
    S = torch.empty(Cout * C * 9, device=dev)
    ws = torch.zeros(vgc.vgc_sqgrad_conv_exact_workspace_bytes(B, C, H, H, Cout, 3, 3, 1, 1, 1, 1), dtype=torch.uint8, device=dev)
    for _ in range(2):
        vgc.vgc_sqgrad_conv_exact(x, d, (3, 3), (1, 1), (1, 1), 1.0, S, ws=ws)
    print(json.dumps({"case": "sqgrad_conv_exact: 3x3 layer-3 shape, per-example statistic", "B": B}))
    for B, n_in, n_out, what in ((32, 2048, 1000, "tensor cores (fc of ResNet-50)"), (8, 1000, 333, "CUDA cores (batch < 32)")):
        x = torch.randn(B, n_in, device=dev); d = torch.randn(B, n_out, device=dev)
        S = torch.empty(n_out * n_in, device=dev)
        ws = torch.zeros(vgc.vgc_sqgrad_linear_workspace_bytes(B, n_in, n_out), dtype=torch.uint8, device=dev)
        for _ in range(2):
            vgc.vgc_sqgrad_linear(x, d, 1.0, S, ws=ws)
        print(json.dumps({"case": "sqgrad_linear: " + what, "B": B, "in": n_in, "out": n_out}))
    # flat buffer: compress, hybrid compress, decode (dense and sparse), index coder
    n, K = 1 << 24, 16
    offs = np.linspace(0, n, K + 1).astype(np.uint32)
    offs_dev = vgc.offsets_tensor(offs)
    g, s = workloads.per_parameter_gs(n, 64, 1e-4, 11, dev)
    r = torch.zeros(n, device=dev); v = torch.zeros(n, device=dev)
    out = vgc.MessageBuffers(n, K, n)
    ws = torch.empty(max(vgc.vgc_compress_workspace_bytes(n, K), vgc.vgc_compress_hybrid_workspace_bytes(n)), dtype=torch.uint8, device=dev)
    for _ in range(2):
        vgc.vgc_compress(g, s, r, v, offs_dev, 2.0, ZETA, out, ws)
    torch.cuda.synchronize()
    c = out.read()
    print(json.dumps({"case": "compress", "n": n, "n_criterion": c["n_criterion"], "nnz": c["nnz"]}))
    hout = vgc.HybridMessageBuffers(n, n)
    r.zero_(); v.zero_()
    tau = float(s.sqrt().median().item())
    for _ in range(2):
        vgc.vgc_compress_hybrid(g, s, r, v, 2.0, ZETA, tau, hout, ws)
    torch.cuda.synchronize()
    print(json.dumps({"case": "compress_hybrid", "n": n, "nnz": hout.read()["nnz"]}))
    u = torch.zeros(n, device=dev); status = torch.zeros(1, dtype=torch.int32, device=dev)
    for density, W in ((0.1, 4), (1e-3, 4)):
        msgs = [workloads.random_message(n, offs, density, 50 + w, dev) for w in range(W)]
        triples = [(m[0], torch.tensor([m[0].numel()], dtype=torch.int32, device=dev), m[1]) for m in msgs]
        for _ in range(2):
            vgc.vgc_decode_accumulate(triples, offs_dev, 1.0 / W, u, status)
            vgc.vgc_decode_sum(triples, offs_dev, 1.0 / W, u, status)
        torch.cuda.synchronize()
        print(json.dumps({"case": "decode_accumulate + decode_sum", "n": n, "W": W, "density": density,
                          "sum_nnz": sum(m[0].numel() for m in msgs)}))
    packed = torch.empty(vgc.vgc_pack_bound_bytes(out.words.numel()), dtype=torch.uint8, device=dev)
    pws = torch.empty(vgc.vgc_pack_workspace_bytes(out.words.numel()), dtype=torch.uint8, device=dev)
    nbytes = torch.zeros(1, dtype=torch.int32, device=dev)
    back = torch.empty_like(out.words)
    for _ in range(2):
        vgc.vgc_pack_indices(out.words, out.counters[0:1], packed, nbytes, status, pws)
        vgc.vgc_unpack_indices(packed, out.counters[0:1], back, status)
    torch.cuda.synchronize()
    print(json.dumps({"case": "pack_indices + unpack_indices", "words": c["nnz"], "packed_bytes": int(nbytes.item())}))


# ----------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline and --impl reference)
# ----------------------------------------------------------------------------------------------
def oracle_sample_time(name: str, n_params: int = 1 << 25):
    """Times the oracle, as it stands, on a bounded sample of the workload.  Returns
    (estimated seconds per full step, description, threads)."""
    import oracle
    from paper_1802_06058_b200 import workloads
    cfg, table, B, x_kind, delta_std, W, alpha = WORKLOADS[name]
    if table is None:
        layers, offsets = [], np.linspace(0, n_params, 17).astype(np.uint32)
    else:
        layers = getattr(workloads, table)()
        offsets = workloads.group_offsets(layers)
    n = int(offsets[-1])
    rng = np.random.default_rng(0)
    # compress + decode at full size on noise inputs (one step each)
    g = rng.standard_normal(n, dtype=np.float32)
    s = (rng.standard_normal(n, dtype=np.float32) ** 2)
    r = np.zeros(n, np.float32); v = np.zeros(n, np.float32)
    t0 = time.perf_counter()
    msg = oracle.compress(g, s, r, v, offsets, alpha, ZETA, want_mask=False)
    t_compress = time.perf_counter() - t0
    t_decode = 0.0
    if W:
        u = np.zeros(n, np.float32)
        t0 = time.perf_counter()
        oracle.decode_accumulate([(msg.words, msg.group_exp)], offsets, 1.0 / W, u)
        t_decode = (time.perf_counter() - t0) * W
    # sqgrad: measure multiply-add rate on a few layers at reduced batch, extrapolate by MAC count
    t_sq, desc = 0.0, ""
    if layers and name != "vgg16":
        total_macs = sum(np.prod(l.gemm_mnk(B)) for l in layers)
        picks = layers if len(layers) <= 3 else [layers[i] for i in (2, 12, len(layers) // 2, 40, len(layers) - 2)]
        bs = B if len(layers) <= 3 else 2
        macs, secs = 0, 0.0
        for li, spec in enumerate(picks):
            x, d = workloads.layer_inputs(spec, bs, cfg, 0, 0, li, x_kind, delta_std, "cpu")
            t0 = time.perf_counter()
            if spec.kind == "conv":
                oracle.sqgrad_conv(x.numpy(), d.numpy(), (spec.k, spec.k), (spec.stride, spec.stride),
                                   (spec.pad, spec.pad), scale=1.0)
            else:
                oracle.sqgrad_linear(x.numpy(), d.numpy(), scale=1.0)
            secs += time.perf_counter() - t0
            macs += int(np.prod(spec.gemm_mnk(bs)))
        t_sq = total_macs / (macs / secs)
        desc = (f"sqgrad: {len(picks)} layers ({', '.join(p.name for p in picks)}) at batch {bs}, "
                f"{macs / secs / 1e9:.2f} GMAC/s extrapolated to {total_macs / 1e9:.1f} GMAC; ")
    desc += f"compress at full n={n} ({t_compress:.2f} s)"
    if W:
        desc += f"; decode of one message x W={W} ({t_decode:.2f} s)"
    return t_sq + t_compress + t_decode, desc, 1, n


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    for i in range(args.warmup + args.steps):
        sec, desc, threads, n = oracle_sample_time(args.workload, args.n_params)
        if i >= args.warmup:
            times.append(sec)
    sec = statistics.mean(times)
    value = n / sec / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "n_params": n},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
def max_over_ranks(value: float, device="cpu") -> float:
    """Largest value over all ranks of the default process group (identity without one)."""
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="resnet50", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="vgc", choices=["vgc", "reference"])
    ap.add_argument("--n-params", type=int, default=1 << 25, help="size of the 'flat' workload")
    ap.add_argument("--per-layer", action="store_true", help="print per-layer sqgrad times instead of the bench line")
    ap.add_argument("--mma-rates", action="store_true",
                    help="print the measured time of one tcgen05.mma instruction per shape (the tensor-pipe ceiling "
                         "the sqgrad kernel is bounded by) instead of the bench line")
    ap.add_argument("--profile-kernels", action="store_true",
                    help="run every kernel form once on a small case and exit (what the ncu captures of profiles/ run)")
    ap.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a CUDA graph")
    ap.add_argument("--streams", type=int, default=5, help="streams the independent sqgrad layers are spread over")
    ap.add_argument("--fused", action="store_true",
                    help="sqgrad adds its sums straight into v and vgc_compress runs without s (12 B read per parameter)")
    ap.add_argument("--algorithm", default="basic", choices=["basic", "hybrid"],
                    help="hybrid: Algorithm 2 (fixed threshold tau + variance criterion) for the compress and decode "
                         "sections; device-timed only (no end-to-end or CPU leg)")
    ap.add_argument("--no-batch", action="store_true",
                    help="one library call per layer instead of one per group of same-shaped conv layers")
    ap.add_argument("--exact-conv", action="store_true",
                    help="conv layers through vgc_sqgrad_conv_exact_batch (per-example statistic); "
                         "device-timed only")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip what the default single-GPU run adds outside the timed steps: the oracle parity check, the "
                         "TF32 peak measurement with the 2-second sqgrad timing, and the config-4 / config-5 sections")
    ap.add_argument("--parity-samples", type=int, default=256,
                    help="entries per layer (at least; one per 128 x 128 tile always) of the squared-gradient sums "
                         "compared with the oracle in the parity check")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the hot path")
    torch.cuda.set_device(local_rank)
    if dist_on:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    import paper_1802_06058_b200 as vgc
    if args.mma_rates:
        if rank == 0:
            import ctypes
            from paper_1802_06058_b200 import _build
            probe = ctypes.CDLL(_build.build_probe())
            probe.vgc_probe_mma_rate.argtypes = [ctypes.c_int] * 6 + [ctypes.POINTER(ctypes.c_double)] * 2
            sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
            for kind, name in ((0, "tf32 (8 k)"), (1, "bf16 (16 k)")):
                for m_rows, a_tmem in ((128, False), (128, True), (64, False)):
                    for n_cols in (64, 128, 256):
                        cyc, tf = ctypes.c_double(0.0), ctypes.c_double(0.0)
                        rc = probe.vgc_probe_mma_rate(kind, int(a_tmem), m_rows, n_cols, 4096, sms, ctypes.byref(cyc), ctypes.byref(tf))
                        print(json.dumps({"operands": name, "A_from": "tensor memory" if a_tmem else "shared memory",
                                          "M": m_rows, "N": n_cols, "status": rc, "cycles_per_mma": round(cyc.value, 1),
                                          "tflops_all_sms": round(tf.value, 1)}))
        return
    vgc.load_library()
    if args.profile_kernels:
        if rank == 0:
            profile_kernels()
        return
    pk = peaks()
    hp = HotPath(args.workload, worker=rank * 16, n_input_sets=2, n_g_sets=max(4, min(args.steps + args.warmup, 16)),
                 n_params=args.n_params, n_streams=1 if args.per_layer else max(args.streams, 1), algorithm=args.algorithm,
                 batch_layers=not args.no_batch, exact_conv=args.exact_conv)
    if args.exact_conv:
        args.no_e2e = True
    if hp.hybrid:
        args.no_e2e = args.no_cpu_baseline = True
    hp.fused = args.fused
    torch.cuda.synchronize()

    if args.per_layer:
        rows = hp.per_layer_times()
        for row in rows:
            print(json.dumps(row))
        print(json.dumps({"total_ms": sum(r["ms"] for r in rows)}))
        return

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, sq, co, de, launches = run_device_timed(hp, args.steps, max(args.warmup, 3), dist_on,
                                                      use_graph=not args.no_graph)
    clocks = sampler.stop()
    counters = hp.out.read()
    if hp.hybrid:
        counters.update(n_criterion=counters["nnz"], n_dropped=0)
    ms_per_step = total_ms / args.steps
    ms_per_step = max_over_ranks(ms_per_step, "cuda")

    n = hp.n
    value = world * n / (ms_per_step * 1e-3) / 1e9
    sq_ms, co_ms, de_ms = statistics.mean(sq), statistics.mean(co), statistics.mean(de)
    nnz_a, nnz = counters["n_criterion"], counters["nnz"]
    sum_nnz = nnz + sum(int(o.words.numel()) for o in hp.others) if hp.W else 0
    compress_bytes = 24 * n + 8 * nnz_a + 4 * nnz
    if hp.hybrid:                                          # the staged word is written, read and written again
        compress_bytes = 24 * n + 12 * nnz
    # decode (vgc_decode_sum): 4 B per word + one write of u
    decode_bytes = (4 * sum_nnz + 4 * n) if hp.W else 0
    gbs = lambda nbytes, ms: nbytes / (ms * 1e-3) / 1e9 if ms > 0 else None
    cd_gbs = gbs(compress_bytes + decode_bytes, co_ms + de_ms)
    sections = {
        "sqgrad_ms": sq_ms, "compress_ms": co_ms, "decode_ms": de_ms,
        "sqgrad_useful_tflops": hp.flops_useful / (sq_ms * 1e-3) / 1e12 if sq_ms > 0 and hp.flops_useful else None,
        "compress_gparam_s": n / (co_ms * 1e-3) / 1e9,
        "compress_gbs": gbs(compress_bytes, co_ms),
        "compress_frac_of_measured_hbm": gbs(compress_bytes, co_ms) / pk["hbm_gbs"],
        "compress_frac_of_8tbs": gbs(compress_bytes, co_ms) / HBM_NOMINAL_GBS,
        "decode_gelem_s": sum_nnz / (de_ms * 1e-3) / 1e9 if hp.W else None,
        "decode_gbs": gbs(decode_bytes, de_ms) if hp.W else None,
        "decode_frac_of_measured_hbm": gbs(decode_bytes, de_ms) / pk["hbm_gbs"] if hp.W else None,
        "decode_frac_of_8tbs": gbs(decode_bytes, de_ms) / HBM_NOMINAL_GBS if hp.W else None,
        "compress_decode_gparam_s": n / ((co_ms + de_ms) * 1e-3) / 1e9,
        # the figure the 70 % target is stated on, against both denominators
        "compress_decode_gbs": cd_gbs,
        "compress_decode_frac_of_measured_hbm": cd_gbs / pk["hbm_gbs"],
        "compress_decode_frac_of_8tbs": cd_gbs / HBM_NOMINAL_GBS,
        "send_density": nnz_a / n, "nnz": nnz, "n_dropped": counters["n_dropped"], "sum_nnz_decoded": sum_nnz,
        "dev_status": counters["dev_status"],
    }
    if args.fused:
        # replayed on their own the sections cannot share v the way the fused step does (the sums would be added
        # without the compressor's reset in between), so the split is taken in the unfused form; the step is fused
        sections["note"] = "section split measured in the unfused form (s written, then read by compress); ms_per_step is the fused step"
    traffic = ncu_traffic()
    compress_traffic = traffic.get("compress_bytes_per_param")
    compress_roofline = {"kernel": "compress_phase_a + compress_count + compress_emit", "bound": "hbm",
                         "achieved": gbs(compress_bytes, co_ms), "peak": pk["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs(compress_bytes, co_ms) / pk["hbm_gbs"],
                         "frac_of_8tbs": gbs(compress_bytes, co_ms) / HBM_NOMINAL_GBS,
                         "traffic": compress_traffic * n if compress_traffic else None,
                         "traffic_source": traffic.get("source"),
                         "algorithmic_bytes": compress_bytes, "peak_source": f"{pk['source']} copy bandwidth, of measured"}
    decode_roofline = None
    if hp.W:
        decode_roofline = {"kernel": "decode_tiles (vgc_decode_sum)", "bound": "hbm", "achieved": gbs(decode_bytes, de_ms),
                           "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": gbs(decode_bytes, de_ms) / pk["hbm_gbs"],
                           "frac_of_8tbs": gbs(decode_bytes, de_ms) / HBM_NOMINAL_GBS,
                           "traffic": traffic.get("decode_bytes_resnet50_w8") if args.workload == "resnet50" and hp.W == 8 else None,
                           "traffic_source": traffic.get("source"), "algorithmic_bytes": decode_bytes,
                           "peak_source": f"{pk['source']} copy bandwidth, of measured"}
    extras = rank == 0 and world == 1 and not args.no_extra
    # dominant kernel of the step
    if sq_ms >= co_ms + de_ms and hp.flops_useful:
        # The contraction must be fp32-accurate (1e-5): three tensor-core products per algorithmic product (hi*hi in
        # TF32 plus two cross terms -- TF32, or bf16 at half the TF32 cost in the TMA-fed form).  issue_factor is their
        # flop-weighted cost in TF32 products; issued = issue_factor x algorithmic is what the tensor pipe is asked to
        # do, and frac = issued / TF32 peak is the load on the pipe.
        issue_factor = hp.flops_issued / hp.flops_useful
        ach_burst = hp.flops_useful / (sq_ms * 1e-3) / 1e12
        roofline = {"kernel": "sqgrad_tc (all layers of one step)", "bound": "tensor", "unit": "TFLOP/s",
                    "issue_factor": issue_factor,
                    "traffic": traffic.get("sqgrad_pass_bytes_resnet50") if args.workload == "resnet50" else None,
                    "traffic_source": traffic.get("source")}
        if extras:
            # the denominators, measured here: cuBLAS TF32 matmul, burst and sustained
            tf32_burst, tf32_sustained = measure_tf32_peak()
            # the numerator in the sustained regime: the sqgrad pass replayed for >= 2 s with the clocks sampled
            sus_ms, sus_clocks = sustained_sqgrad(hp, local_rank, seconds=2.0)
            ach = hp.flops_useful / (sus_ms * 1e-3) / 1e12
            roofline.update({
                "achieved": ach, "peak": tf32_sustained / issue_factor, "frac": issue_factor * ach / tf32_sustained,
                "regime": "sustained: sqgrad pass replayed back to back for >= 2 s, against the TF32 matmul rate sustained "
                          "over 2 s (both under the power cap)",
                "sqgrad_ms_sustained": sus_ms, "clocks_sustained": sus_clocks,
                "issued_tflops": issue_factor * ach, "algorithmic_frac": ach / tf32_sustained,
                "tf32_peak_sustained": tf32_sustained, "tf32_peak_burst": tf32_burst,
                "burst": {"sqgrad_ms": sq_ms, "achieved": ach_burst, "issued_tflops": issue_factor * ach_burst,
                          "frac": issue_factor * ach_burst / tf32_burst, "algorithmic_frac": ach_burst / tf32_burst,
                          "regime": "burst: a few graph replays at the clocks of `clocks`, against the best of 10 single matmuls"},
                "peak_source": "TF32 torch.matmul 8192^3 measured in this run (best of 10 = burst, back to back for 2 s = "
                               "sustained), the way MEASURED_PEAKS.json measures bf16; of measured",
                "bf16_half_for_reference": {"burst": pk["bf16_tflops"] / 2.0, "sustained": pk["bf16_tflops_sustained"] / 2.0,
                                            "source": pk["source"]}})
        else:
            tf32_peak = pk["bf16_tflops"] / 2.0                # nominal tf32 : bf16 ratio is 1 : 2
            roofline.update({"achieved": ach_burst, "peak": tf32_peak / issue_factor,
                             "frac": issue_factor * ach_burst / tf32_peak, "issued_tflops": issue_factor * ach_burst,
                             "algorithmic_frac": ach_burst / tf32_peak, "regime": "burst",
                             "peak_source": f"{pk['source']} bf16 burst x 1/2 (tf32 nominal ratio), of measured"})
        roofline["note"] = ("achieved = algorithmic flops 2*M*N*K per layer / sqgrad time; peak = TF32 peak / issue_factor; "
                            "frac = issued TF32-equivalent flops / TF32 peak (pipe load); algorithmic_frac = achieved / TF32 peak")
    else:
        roofline = compress_roofline
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 (split into tf32 hi*hi + tf32 or bf16 cross terms on the tensor cores)",
            "data": "synthetic",
            "config": {"workload": args.workload, "n_params": n, "batch": hp.batch, "W": hp.W, "alpha": hp.alpha,
                       "zeta": ZETA, "groups": hp.K, "algorithm": args.algorithm, "tau": hp.tau, "launch": "eager" if args.no_graph else "cuda graph replay",
                       "sqgrad_streams": getattr(hp, "n_streams", 1), "input_sets_rotated": len(hp.inputs),
                       "sqgrad_calls": len(getattr(hp, "groups", [])), "conv_statistic": "per-example" if args.exact_conv else "per-position",
                       "fused_sqgrad_into_v": bool(args.fused),
                       "l2": "inputs larger than L2 (no flush)" if n * 16 > 126e6 else "state fits in L2 (no flush): cache-resident numbers"},
            "gpu_launches": int(launches), "clocks": clocks, "sections": sections, "roofline": roofline,
            "roofline_compress": compress_roofline, "roofline_decode": decode_roofline}

    if not args.no_e2e:
        e2e_ms, h2d, d2h = run_e2e(hp, min(args.steps, 5), 1)
        e2e_ms = max_over_ranks(e2e_ms, "cuda")
        line["e2e"] = {"value": world * n / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)}
    if extras and not args.exact_conv and not args.fused:
        # one more step of exactly what was timed, against the oracle (outside every timed region)
        line["parity"] = parity_check(hp, sqgrad_samples=args.parity_samples)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, desc, threads, _ = oracle_sample_time(args.workload, args.n_params)
        line["cpu_baseline"] = {"value": n / sec / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": desc, "host_cores_available": os.cpu_count()}
    if extras and args.workload == "resnet50" and not hp.hybrid:
        del hp
        torch.cuda.empty_cache()
        line["config4"] = config4_compress(pk)
        line["config5"] = config5_decode_sweep(pk)
    if rank == 0:
        print(json.dumps(line))
    if dist_on:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
