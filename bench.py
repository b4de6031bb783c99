#!/usr/bin/env python
"""Benchmark of the in-hindsight int8 layer path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: every layer call
of the workload (tensor-core implicit GEMM or depthwise kernel with the fused requantization +
min/max epilogue) followed by one range update for all of the workload's tensors.  The metric is
int8 tera-operations per second (2 x MACs of the dense definition) of the in-hindsight path; the
same run also times the dynamic-quantization comparison path and reports algorithmic HBM bytes
per layer for both (Eq. 4 / Eq. 5 of arxiv 2105.04246).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg1|cfg3|cfg4|cfg5]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

Prints ONE JSON line on rank 0.
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

from paper_2105_04246_b200 import synth
from paper_2105_04246_b200 import workloads as wl

METRIC = "int8 TOPS & HBM bytes/layer: hindsight-fused vs dynamic quant, % of roofline"
NOMINAL_INT8_OVER_BF16 = 2.0          # dense int8 peak / dense bf16 peak on B200 (4.5 / 2.25 POPS)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the named layer's kernel: mean over the last 16 of 24
# launches that rotate over a buffer pool larger than L2, caches not flushed between launches, so that the output of
# earlier launches is written back to DRAM while later ones run (ncu captures summarised under profiles/, taken with
# the kernels as committed; set an entry to None when its kernel changes).
NCU_TRAFFIC = {
    "stem7x7": 122226672, "layer1.0": 50976208, "layer2.1": 25329152, "layer3.1": 12603200, "layer4.1": 6623488,
    "resnet_conv3x3_64": 25385552, "resnet_conv3x3_256_bwd": 25491936,
    "mbv2_expand": 135021248, "mbv2_dw3x3": 231826688, "mbv2_project": 135043808,
}
# kernels other than the tensor-core layer kernel, by layer name
KERNEL_OF = {"mbv2_dw3x3": "depthwise3x3_col_kernel", "stem7x7": "hq_gather_conv_kernel"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ---- workloads ---------------------------------------------------------------------------------
def workload_layers(name: str, batch_div: int = 1):
    """[(kind, shape, input recipe)] in call order; chained=True feeds each output to the next layer."""
    def b(s):
        return s.with_batch(max(1, s.N // batch_div)) if batch_div > 1 else s
    if name == "cfg1":
        return [("linear", wl.CFG1_LINEAR, "uniform")], False
    if name == "cfg2":
        return [("conv_fwd", b(wl.CFG2_CONV), "relu")], False
    if name == "cfg3":
        return [("conv_bwd", b(wl.CFG3_BWD), "grad")], False
    if name == "cfg4":
        return [("conv_fwd", b(wl.CFG4_EXPAND), "signed"), ("conv_fwd", b(wl.CFG4_DW), None), ("conv_fwd", b(wl.CFG4_PROJECT), None)], True
    if name == "cfg4b":
        # backward data through the same inverted residual, last layer first; each input gradient feeds the layer before
        return [("conv_bwd", b(wl.CFG4_PROJECT), "grad"), ("conv_bwd", b(wl.CFG4_DW), None), ("conv_bwd", b(wl.CFG4_EXPAND), None)], True
    if name == "cfg5":
        # every convolution of ResNet-18 at 224x224 and the classifier, forward and backward-data (none for the stem);
        # each call has its own synthetic input: what sits between the layers (BN, ReLU, pooling, adds) is not on the path
        convs, fc = wl.resnet18_layers(max(1, 128 // batch_div))
        fwd = [("conv_fwd", c, "image" if c.C == 3 else "relu") for c in convs] + [("linear", fc, "relu")]
        fc_bwd = wl.LinearShape("fc.bwd", fc.M, fc.K, fc.N)
        bwd = [("conv_bwd", wl.replace(c, name=c.name + ".bwd"), "grad") for c in convs[1:]] + [("linear", fc_bwd, "grad")]
        return fwd + bwd, False
    raise SystemExit(f"unknown workload {name}")


def make_input(recipe: str, g, shape):
    if recipe == "uniform":
        return synth.uniform_int8(g, shape, scale=0.02)
    if recipe == "relu":
        return synth.tiled(synth.relu_activations, g, shape)
    if recipe == "signed":
        return synth.tiled(synth.signed_activations, g, shape)
    if recipe == "grad":
        return synth.tiled(synth.gradients, g, shape)
    if recipe == "image":
        return synth.tiled(synth.image_like, g, shape)
    raise ValueError(recipe)


def layer_shapes(kind, s):
    """(input shape, output shape, weight shape)"""
    if kind == "linear":
        return (s.M, s.K), (s.M, s.N), (s.N, s.K)
    wshape = (s.K, s.R, s.S) if s.depthwise else (s.K, s.R, s.S, s.C)
    x, y = (s.N, s.H, s.W, s.C), (s.N, s.Ho, s.Wo, s.K)
    return (x, y, wshape) if kind == "conv_fwd" else (y, x, wshape)


# ---- reference arm: the CPU oracle, as it stands --------------------------------------------------
def oracle_step(kind, s, x, w, layer):
    import oracle as O
    if kind == "linear":
        acc = O.linear_acc(x.q, x.zero_point, w.q)
    else:
        d = O.conv_desc(s.N, s.H, s.W, s.C, s.K, s.R, s.S, s.stride, s.pad, s.groups)
        acc = O.conv_fwd_acc(d, x.q, x.zero_point, w.q) if kind == "conv_fwd" else O.conv_bwd_data_acc(d, x.q, x.zero_point, w.q)
    return layer.step(acc, O.acc_scale(x.scale, w.scale))


def run_oracle(workload: str, steps: int, warmup: int, budget_s: float):
    """Times the oracle on a bounded sample of the workload: the same layers at a reduced batch."""
    import oracle as O
    O.build()
    cores = os.cpu_count() or 1
    full, chained = workload_layers(workload)
    full_ops = sum(s.ops for _, s, _ in full)
    # sample: shrink the batch so that one step is roughly budget_s / (steps + warmup) of CPU work at ~10 GOP/s
    per_step_ops = max(2e8, budget_s / max(1, steps + warmup) * 1.0e10)
    div = 1
    while full_ops / div > per_step_ops and div < 256 and workload != "cfg1":
        div *= 2
    layers, _ = workload_layers(workload, div)
    g = synth.rng(77, div)
    ws, xs, ls = [], [], []
    for kind, s, recipe in layers:
        xsh, _, wsh = layer_shapes(kind, s)
        ws.append(synth.weights(g, wsh) if kind != "linear" else synth.uniform_int8(g, wsh, scale=0.01))
        xs.append(make_input(recipe, g, xsh) if recipe else None)
        ls.append(O.Layer(0.9))
    ops = sum(s.ops for _, s, _ in layers)

    def one_step():
        prev = None
        for i, (kind, s, _) in enumerate(layers):
            x = xs[i] if xs[i] is not None else prev
            res = oracle_step(kind, s, x, ws[i], ls[i])
            st = ls[i].state
            prev = synth.QTensor(res.q, st.scale, st.zero_point)

    for _ in range(warmup):
        one_step()
    t0 = time.perf_counter()
    for _ in range(steps):
        one_step()
    dt = time.perf_counter() - t0
    sample = f"{workload} layers at batch/{div} ({ops / 1e9:.3f} GOP per step), {steps} steps, oracle accumulate + min/max + quantize + range update"
    return ops * steps / dt / 1e12, dt / steps * 1e3, cores, sample


# ---- GPU arm ---------------------------------------------------------------------------------------
L2_ROTATE_BYTES = 192 << 20           # per-layer buffer pools are sized so that one cycle through them moves more than L2 (126 MB)
MAX_POOL = 64


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi every 50 ms while timed regions run."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag = index, [], False

    def run(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        while not self.stop_flag:
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits"],
                                     capture_output=True, text=True, timeout=5).stdout.strip()
                if out:
                    self.samples.append((time.perf_counter(), [v.strip() for v in out.split(",")]))
            except Exception:
                pass
            time.sleep(0.05)

    def summary(self, t0: float | None = None, t1: float | None = None):
        rows = [s for (t, s) in self.samples if (t0 is None or t >= t0) and (t1 is None or t <= t1)]
        sm = [float(s[0]) for s in rows if s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in rows if s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for s in rows for i in range(4) if len(s) >= 6 and s[2 + i].lower().startswith("active")})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None, "reasons": reasons,
                "samples": len(rows)}


class GpuWorkload:
    """All device buffers of one workload plus the calls of one step (hindsight or dynamic).

    Every layer has its own pool of input / output / workspace buffer sets, sized so that one cycle through the pool
    moves more bytes than the L2 holds: back-to-back launches of ONE layer then meet cold operands, as they do inside a
    whole step (where the other layers' traffic flushes the cache)."""

    def __init__(self, name: str, ctx, dev, seed_key: int, stochastic: bool = False, pool_cap: int = MAX_POOL):
        import torch
        from paper_2105_04246_b200 import hq
        self.hq, self.torch, self.ctx, self.dev, self.name = hq, torch, ctx, dev, name
        self.layers, self.chained = workload_layers(name)
        n = len(self.layers)
        g = synth.rng(1000 + seed_key)
        st = hq.new_states(n)
        if stochastic:                      # the paper's rounding for gradients: backward-data layers only
            for i, (kind, _s, _r) in enumerate(self.layers):
                if kind == "conv_bwd" or _s.name.endswith(".bwd"):
                    st[i]["rounding"], st[i]["seed"] = hq.ROUND_STOCHASTIC, 0x2105 + i
        self.states = hq.states_to_device(st, dev)
        self.state_ptr = [self.states.data_ptr() + hq.STATE_BYTES * i for i in range(n)]
        self.W, self.w_scale, self.pw, self.desc, self.x_pool, self.xq_pool, self.y_pool, self.ws_pool, self.pool = [], [], [], [], [], [], [], [], []
        stream = torch.cuda.current_stream(dev)
        for i, (kind, s, recipe) in enumerate(self.layers):
            xsh, ysh, wsh = layer_shapes(kind, s)
            xb, yb = int(np.prod(xsh)), int(np.prod(ysh))
            pool = 2 if self.chained else int(min(pool_cap, max(2, -(-L2_ROTATE_BYTES // (xb + yb)))))
            self.pool.append(pool)
            w = synth.weights(g, wsh) if kind != "linear" else synth.uniform_int8(g, wsh, scale=0.01)
            self.W.append(torch.from_numpy(w.q).to(dev))
            self.w_scale.append(torch.tensor([w.scale], dtype=torch.float32, device=dev))
            if kind == "linear":          # weights prepared once: padded copy and column sums cached, one launch per call
                self.desc.append(None)
                self.pw.append(ctx.linear_prepare(stream, s.N, s.K, self.W[-1], 0, s.M))
            else:
                d = hq.conv_desc(s.N, s.H, s.W, s.C, s.K, s.R, s.S, s.stride, s.pad, s.groups)
                self.desc.append(d)
                self.pw.append(ctx.weights_prepare(stream, d, hq.DIR_FWD if kind == "conv_fwd" else hq.DIR_BWD_DATA, self.W[-1]))
            if recipe is not None:
                xs, xqs = [], []
                base = make_input(recipe, g, xsh)
                base_d = torch.from_numpy(np.ascontiguousarray(base.q)).to(dev)
                for j in range(pool):
                    # pool members: the same samples rolled by a prime offset (distinct bytes at every address)
                    xs.append(base_d if j == 0 else torch.roll(base_d.reshape(-1), 104729 * j).reshape(xsh).contiguous())
                    xqs.append(hq.states_to_device(hq.input_state(base.scale * (1.0 + 0.05 * (j % 3)), base.zero_point), dev))
                self.x_pool.append(xs)
                self.xq_pool.append(xqs)
            else:
                self.x_pool.append(None)
                self.xq_pool.append(None)
            self.y_pool.append([torch.empty(ysh, dtype=torch.int8, device=dev) for _ in range(pool)])
            self.ws_pool.append(None)
        self.ops = sum(s.ops for _, s, _ in self.layers)
        self.static_bytes = [wl.layer_static_bytes(s, kind == "conv_bwd" or s.name.endswith(".bwd")) for kind, s, _ in self.layers]
        self.dynamic_bytes = [wl.layer_dynamic_bytes(s, kind == "conv_bwd" or s.name.endswith(".bwd")) for kind, s, _ in self.layers]
        self.h2d_bytes = sum(int(np.prod(layer_shapes(k, s)[0])) for (k, s, r) in self.layers if r is not None)
        self.d2h_bytes = int(np.prod(layer_shapes(*self.layers[-1][:2])[1]))

    def _inputs(self, i, j):
        if self.x_pool[i] is not None:
            jj = j % self.pool[i]
            return self.x_pool[i][jj], self.xq_pool[i][jj].data_ptr()
        return self.y_pool[i - 1][j % self.pool[i - 1]], self.state_ptr[i - 1]

    def layer_call(self, stream, i, j, dynamic=False):
        hq, ctx = self.hq, self.ctx
        kind, s, _ = self.layers[i]
        x, xq = self._inputs(i, j)
        y = self.y_pool[i][j % self.pool[i]]
        if dynamic:
            if self.ws_pool[i] is None:   # the binary32 intermediate of Eq. 5 rotates like the other buffers
                nws = int(min(self.pool[i], max(2, -(-L2_ROTATE_BYTES // (4 * y.numel())))))
                self.ws_pool[i] = [self.torch.empty(y.shape, dtype=self.torch.float32, device=self.dev) for _ in range(nws)]
            ws = self.ws_pool[i][j % len(self.ws_pool[i])]
            if kind == "linear":
                op = hq.linear_op(s.M, s.N, s.K, x, xq, self.W[i], self.w_scale[i], pw=self.pw[i])
            else:
                op = hq.conv_op(hq.OP_CONV_FWD if kind == "conv_fwd" else hq.OP_CONV_BWD_DATA, self.desc[i], x, xq, self.pw[i], self.w_scale[i])
            ctx.dynamic_quant(stream, op, ws, y, self.state_ptr[i])
        elif kind == "linear":
            ctx.linear_fwd_prepared(stream, s.M, x, xq, self.pw[i], self.w_scale[i], None, y, self.state_ptr[i])
        elif kind == "conv_fwd":
            ctx.conv_fwd(stream, self.desc[i], x, xq, self.pw[i], self.w_scale[i], y, self.state_ptr[i])
        else:
            ctx.conv_bwd_data(stream, self.desc[i], x, xq, self.pw[i], self.w_scale[i], y, self.state_ptr[i])

    def step(self, stream, j, dynamic=False, only_layer=None, update=True, exchange=None):
        for i in range(len(self.layers)):
            if only_layer is None or only_layer == i:
                self.layer_call(stream, i, j, dynamic)
        if update and not dynamic:
            if exchange is not None:      # batch shards: min/max over all ranks before Eq. 2-3
                exchange(stream, self.states)
            self.ctx.range_update(stream, self.states, len(self.layers), 0.9)

    def release(self):
        for pw in self.pw:
            if pw is not None:
                pw.release()
        self.x_pool = self.y_pool = self.ws_pool = self.W = None


def capture(torch, stream_fn, reps: int):
    """Captures `reps` consecutive steps (pool slot = rep index) into one CUDA graph."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        s = torch.cuda.current_stream()
        for j in range(reps):
            stream_fn(s, j)
    return g


def timed_repeats(torch, run_once, units: int, min_time_s: float, min_repeats: int, dist=None, max_repeats: int = 4000):
    """Runs `run_once` (which enqueues `units` steps or launches) as often as it takes to fill `min_time_s`, at least
    `min_repeats` times, each repeat between its own pair of CUDA events on the launching stream (with more than one rank:
    a barrier and a device synchronisation on both sides of every repeat, and the maximum over the ranks).
    Returns per-unit times in ms: (median, min, max, repeats)."""
    def one():
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_once()
        e1.record()
        if dist is not None:
            torch.cuda.synchronize()
            dist.barrier()
            t = torch.tensor([e0.elapsed_time(e1)], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return (e0, e1)
    torch.cuda.synchronize()
    first = one()
    if dist is None:
        torch.cuda.synchronize()
        first = first[0].elapsed_time(first[1])
    reps = int(min(max_repeats, max(min_repeats, -(-min_time_s * 1e3 // max(first, 1e-3)))))
    if dist is not None:    # every rank must run the same number of repeats
        t = torch.tensor([reps], device="cuda", dtype=torch.int64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        reps = int(t.item())
    got = [one() for _ in range(reps)]
    if dist is None:
        torch.cuda.synchronize()
        got = [a.elapsed_time(b) for (a, b) in got]
    per = sorted(x / units for x in got)
    return statistics.median(per), per[0], per[-1], reps


def measure_mma_peak(torch, ctx, sampler, sustained_s: float = 4.0):
    """int8 MMA-only throughput of this GPU: best of 10 launches (burst) and back-to-back launches for `sustained_s`."""
    out = {}
    chunks = 512                                             # 512 x 32 instructions per SM: about a millisecond
    for pair in (0, 1):
        ops = ctx.mma_peak_probe(None, pair, 256, chunks)    # warm-up
        torch.cuda.synchronize()
        best = None
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.mma_peak_probe(None, pair, 256, chunks)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        out["pair" if pair else "single"] = {"burst_tops": round(ops / (best * 1e-3) / 1e12, 1)}
    pair = 1 if out["pair"]["burst_tops"] >= out["single"]["burst_tops"] else 0
    n = max(1, int(sustained_s * 1e3 / max(best, 1e-3)))
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        ops = ctx.mma_peak_probe(None, pair, 256, chunks)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    sus = ops * n / (e0.elapsed_time(e1) * 1e-3) / 1e12
    clk = sampler.summary(t0 + 0.5, t1)
    assert ctx.get_async_error() == 0, "a device-side wait expired in the MMA probe"
    return {"burst_tops": max(out["pair"]["burst_tops"], out["single"]["burst_tops"]), "single_cta_burst_tops": out["single"]["burst_tops"],
            "cta_pair_burst_tops": out["pair"]["burst_tops"], "sustained_tops": round(sus, 1), "sustained_s": round(t1 - t0, 2),
            "sustained_sm_mhz": clk["sm_mhz"], "sustained_reasons": clk["reasons"],
            "what": "tcgen05.mma kind::i8 128x256x32 (pair: 256x256x32) issued back to back on operand tiles resident in shared memory, every SM, no loads, no epilogue"}


def check_waits(ctx, where: str):
    """Every device-side wait of the kernels is bounded; one that expired leaves a code in the context's status word."""
    code = ctx.get_async_error()
    assert code == 0, f"a device-side wait expired (code {code}) during: {where}"


def layer_rows(torch, wk, cfg_name, peaks, probe_peak, min_time_s, min_repeats):
    """Per-layer rows of one workload: each layer's launches alone (no update kernel), replayed from a CUDA graph that
    cycles through the layer's whole buffer pool; hindsight and dynamic path."""
    int8_peak = peaks["bf16_tflops"] * NOMINAL_INT8_OVER_BF16
    hbm_peak = peaks["hbm_gbs"]
    rows = []
    for i, (kind, s, _) in enumerate(wk.layers):
        reps = wk.pool[i] if not wk.chained else 2
        if wk.chained:
            # a chained layer reads the previous layer's output: make sure every pool slot of that output exists
            g_h = capture(torch, lambda st, j, ii=i: wk.step(st, j, only_layer=ii, update=False), reps)
            g_d = capture(torch, lambda st, j, ii=i: wk.step(st, j, dynamic=True, only_layer=ii), reps)
        else:
            g_h = capture(torch, lambda st, j, ii=i: wk.layer_call(st, ii, j), reps)
            g_d = capture(torch, lambda st, j, ii=i: wk.layer_call(st, ii, j, dynamic=True), reps)
        ms, lo, hi, r = timed_repeats(torch, g_h.replay, reps, min_time_s, min_repeats)
        check_waits(wk.ctx, f"{cfg_name} {s.name} in-hindsight")
        msd, lod, hid, rd = timed_repeats(torch, g_d.replay, reps, min_time_s, min_repeats)
        check_waits(wk.ctx, f"{cfg_name} {s.name} dynamic")
        del g_h, g_d
        us, usd = ms * 1e3, msd * 1e3
        dw = getattr(s, "depthwise", False)
        t_tensor = s.ops / (int8_peak * 1e12) * 1e6
        t_hbm = wk.static_bytes[i] / (hbm_peak * 1e9) * 1e6
        rows.append({
            "config": cfg_name, "layer": s.name, "kind": kind, "us": round(us, 3), "us_min": round(lo * 1e3, 3), "us_max": round(hi * 1e3, 3),
            "repeats": r, "launches_per_repeat": reps, "us_dynamic": round(usd, 3),
            "tops": round(s.ops / us / 1e6, 2), "gbs": round(wk.static_bytes[i] / us / 1e3, 1),
            "gbs_dynamic": round(wk.dynamic_bytes[i] / usd / 1e3, 1),
            "hbm_bytes_hindsight": int(wk.static_bytes[i]), "hbm_bytes_dynamic": int(wk.dynamic_bytes[i]),
            "bound": "alu-or-hbm" if dw else ("tensor" if t_tensor >= t_hbm else "hbm"),
            "frac_tensor": None if dw else round(t_tensor / us, 4),
            "frac_tensor_probe": None if (dw or not probe_peak) else round(s.ops / (probe_peak * 1e12) * 1e6 / us, 4),
            "frac_hbm": round(t_hbm / us, 4),
            "traffic": NCU_TRAFFIC.get(s.name),
        })
    return rows


def spawn_ranks(args) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one per GPU) the way torchrun would."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_gpu(args):
    import torch
    from paper_2105_04246_b200 import hq

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    ctx = hq.Context(local)
    if args.no_overlap:
        ctx.set_option("overlap_launches", 0)
    ctx.set_option("depthwise", args.depthwise)
    peaks, peak_kind = load_peaks()
    name = args.workload
    K, W = args.steps, max(3, args.warmup)
    stream = torch.cuda.current_stream(dev)
    sampler = ClockSampler(local)
    sampler.start()

    # what the tensor cores of this GPU sustain on int8 with nothing else in the way (second denominator of the tensor roofline)
    probe = None
    if not args.no_probe and rank == 0:
        probe = measure_mma_peak(torch, ctx, sampler, sustained_s=args.probe_seconds)
    probe_peak = probe["burst_tops"] if probe else None

    wk = GpuWorkload(name, ctx, dev, seed_key=rank, stochastic=args.rounding == "stochastic")
    n_layers = len(wk.layers)
    cyc = 2                                   # steps per captured graph; a whole step moves far more than L2 by itself

    # iteration 0 of the scheme: the dynamic path initialises every range (also warms the dynamic kernels up)
    for j in range(cyc):
        wk.step(stream, j, dynamic=True)
    torch.cuda.synchronize()
    exchange = None
    if dist is not None:
        from paper_2105_04246_b200 import parallel
        exchange = parallel.StatsExchange(ctx, n_layers, dev)
    l0 = ctx.launch_count()
    wk.step(stream, 0, exchange=exchange)
    launches_per_step = ctx.launch_count() - l0
    torch.cuda.synchronize()

    # graphs: the launch-bound loop is replayed from CUDA graphs (all parameters live in device memory); with several
    # ranks the statistics exchange (pack kernel, NCCL all-reduce, unpack kernel) is part of the captured step
    g_full = capture(torch, lambda s, j: wk.step(s, j, exchange=exchange), cyc)
    g_single = capture(torch, lambda s, j: wk.step(s, j, exchange=exchange), 1)
    g_dyn = capture(torch, lambda s, j: wk.step(s, j, dynamic=True), cyc)
    g_dyn_single = capture(torch, lambda s, j: wk.step(s, j, dynamic=True), 1)

    def k_steps(gf, g1):
        def run():
            for _ in range(K // cyc):
                gf.replay()
            for _ in range(K % cyc):
                g1.replay()
        return run

    for _ in range(-(-W // cyc)):
        g_full.replay()
        g_dyn.replay()
    torch.cuda.synchronize()

    t_sec0 = time.perf_counter()
    ms_step, ms_lo, ms_hi, repeats = timed_repeats(torch, k_steps(g_full, g_single), K, args.min_time, args.min_repeats, dist)
    t_sec1 = time.perf_counter()
    step_clocks = sampler.summary(t_sec0, t_sec1)
    ms_dyn, _, _, _ = timed_repeats(torch, k_steps(g_dyn, g_dyn_single), K, args.min_time, args.min_repeats, dist)

    # per-layer kernel durations of this workload, then of the other configurations (rows only)
    per_layer = layer_rows(torch, wk, name, peaks, probe_peak, args.min_time, args.min_repeats)
    layer_us = [r["us"] for r in per_layer]

    # end to end through the binding with host buffers: every step copies its inputs from pinned host memory, runs, and
    # copies its result back to pinned host memory.  Copies run on their own streams, ordered against the compute stream
    # with events per slot, so the H2D of step k+1 and the D2H of step k-1 overlap step k (as a serving loop would).
    e2e_steps = max(4, min(K, 50))
    host_in = [[xs[j % len(xs)].cpu().pin_memory() for j in range(cyc)] if xs is not None else None for xs in wk.x_pool]
    host_out = [torch.empty(wk.y_pool[-1][0].shape, dtype=torch.int8).pin_memory() for _ in range(cyc)]
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(cyc)]
    ev_done = [torch.cuda.Event() for _ in range(cyc)]
    ev_out = [torch.cuda.Event() for _ in range(cyc)]
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        j = k % cyc
        with torch.cuda.stream(s_in):
            if k >= cyc:
                s_in.wait_event(ev_done[j])          # the step that last read this slot's inputs has finished
            for i in range(n_layers):
                if host_in[i] is not None:
                    wk.x_pool[i][j].copy_(host_in[i][j], non_blocking=True)
            ev_in[j].record(s_in)
        stream.wait_event(ev_in[j])
        if k >= cyc:
            stream.wait_event(ev_out[j])             # the slot's previous result has left the device
        wk.step(stream, j, exchange=exchange)
        ev_done[j].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[j])
            host_out[j].copy_(wk.y_pool[-1][j % wk.pool[-1]], non_blocking=True)
            ev_out[j].record(s_out)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    del host_in, host_out
    code = ctx.get_async_error()
    assert code == 0, f"a device-side wait expired during the benchmark (code {code})"
    if dist is not None:
        t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())

    # the other configurations: per-layer rows and a step value each (rank 0 of a single-GPU run only)
    other = {}
    if args.all_configs and world == 1:
        ops_main, static_main, dyn_main = wk.ops, list(wk.static_bytes), list(wk.dynamic_bytes)
        layers_main = list(wk.layers)
        wk.release()
        del g_full, g_single, g_dyn, g_dyn_single
        torch.cuda.empty_cache()
        for cfg in [c for c in ("cfg1", "cfg2", "cfg3", "cfg4") if c != name]:
            w2 = GpuWorkload(cfg, ctx, dev, seed_key=rank)
            for j in range(2):
                w2.step(stream, j, dynamic=True)
            check_waits(ctx, f"{cfg} first dynamic steps")
            w2.step(stream, 0)
            check_waits(ctx, f"{cfg} first in-hindsight step")
            cyc2 = 2 if w2.chained else max(w2.pool)
            gs = capture(torch, lambda s, j: w2.step(s, j), cyc2)
            gd = capture(torch, lambda s, j: w2.step(s, j, dynamic=True), cyc2)
            for _ in range(3):
                gs.replay(); gd.replay()
            check_waits(ctx, f"{cfg} warm-up replays")
            ms2, lo2, hi2, r2 = timed_repeats(torch, gs.replay, cyc2, args.min_time, args.min_repeats)
            check_waits(ctx, f"{cfg} in-hindsight steps")
            msd2, _, _, _ = timed_repeats(torch, gd.replay, cyc2, args.min_time, args.min_repeats)
            check_waits(ctx, f"{cfg} dynamic steps")
            del gs, gd
            per_layer += layer_rows(torch, w2, cfg, peaks, probe_peak, args.min_time, args.min_repeats)
            other[cfg] = {"workload": f"{cfg}: " + ", ".join(s.name for _, s, _ in w2.layers), "value": round(w2.ops / (ms2 * 1e-3) / 1e12, 3),
                          "unit": "TOPS", "ms_per_step": round(ms2, 6), "ms_per_step_min": round(lo2, 6), "ms_per_step_max": round(hi2, 6),
                          "repeats": r2, "steps_per_repeat": cyc2,
                          "dynamic": {"value": round(w2.ops / (msd2 * 1e-3) / 1e12, 3), "ms_per_step": round(msd2, 6)},
                          "hbm_bytes_per_step": {"hindsight": int(sum(w2.static_bytes)), "dynamic": int(sum(w2.dynamic_bytes))}}
            check_waits(ctx, f"{cfg} layer rows")
            w2.release()
            del w2
            torch.cuda.empty_cache()
        wk_ops, wk_static, wk_dynamic, wk_layers = ops_main, static_main, dyn_main, layers_main
    else:
        wk_ops, wk_static, wk_dynamic, wk_layers = wk.ops, wk.static_bytes, wk.dynamic_bytes, wk.layers
    sampler.stop_flag = True
    sampler.join(timeout=2)

    tops = wk_ops * world / (ms_step * 1e-3) / 1e12
    int8_peak = peaks["bf16_tflops"] * NOMINAL_INT8_OVER_BF16
    hbm_peak = peaks["hbm_gbs"]
    # dominant kernel of the step = the layer with the longest measured launch
    dom = max(range(n_layers), key=lambda i: layer_us[i])
    kind, s, _ = wk_layers[dom]
    t_tensor = s.ops / (int8_peak * 1e12) * 1e6
    t_hbm = wk_static[dom] / (hbm_peak * 1e9) * 1e6
    dw = getattr(s, "depthwise", False)
    if dw or t_hbm > t_tensor:
        ach = wk_static[dom] / layer_us[dom] / 1e3
        roof = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s", "frac": round(ach / hbm_peak, 4),
                "peak_source": f"{peak_kind} copy bandwidth"}
    else:
        ach = s.ops / layer_us[dom] / 1e6
        roof = {"bound": "tensor", "achieved": round(ach, 1), "peak": round(int8_peak, 1), "unit": "TOP/s", "frac": round(ach / int8_peak, 4),
                "peak_source": f"{peak_kind} bf16 burst x {NOMINAL_INT8_OVER_BF16} (nominal int8 / bf16 ratio)",
                "frac_of_mma_probe": None if not probe_peak else round(ach / probe_peak, 4)}
    tr = NCU_TRAFFIC.get(s.name)
    roof.update({"kernel": KERNEL_OF.get(s.name, "depthwise3x3_col_kernel" if dw else "hq_gemm_kernel"), "layer": s.name,
                 "launch_us": round(layer_us[dom], 3), "algorithmic_bytes": int(wk_static[dom]), "traffic": tr,
                 "frac_of": f"of {peak_kind}"})

    out = {
        "metric": METRIC, "value": round(tops, 3), "unit": "TOPS", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(ms_step, 6), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "impl": "hq",
        "config": {"workload": f"{name}: " + ", ".join(s.name for _, s, _ in wk_layers), "path": "in-hindsight (static requant in the epilogue + min/max)",
                   "l2": "every layer's inputs, outputs and workspaces rotate over a pool of buffer sets whose cycle moves more than L2 (192 MB); "
                         "a whole step moves about 1 GB",
                   "eta": 0.9,
                   "launch": "ordinary" if args.no_overlap else "programmatic stream serialization",
                   "rounding": "nearest even" if args.rounding == "nearest" else "stochastic for gradient layers, nearest even otherwise",
                   "parallelism": f"dp{world} (batch shards; one int32 min/max all-reduce per step before the range update, inside the captured step)" if world > 1 else "dp1"},
        "timing": {"repeats": repeats, "steps_per_repeat": K, "ms_per_step_min": round(ms_lo, 6), "ms_per_step_max": round(ms_hi, 6),
                   "min_time_s": args.min_time, "statistic": "median over repeats; each repeat is exactly `steps` steps between its own CUDA events",
                   "sm_mhz_during_steps": step_clocks["sm_mhz"],
                   "ms_per_step_x_sm_mhz": None if not step_clocks["sm_mhz"] else round(ms_step * step_clocks["sm_mhz"], 3)},
        "gpu_launches": int(launches_per_step * K * repeats),
        "launches_per_step": int(launches_per_step),
        "dynamic": {"value": round(wk_ops * world / (ms_dyn * 1e-3) / 1e12, 3), "unit": "TOPS", "ms_per_step": round(ms_dyn, 6)},
        "hbm_bytes_per_step": {"hindsight": int(sum(wk_static)), "dynamic": int(sum(wk_dynamic))},
        "layers": per_layer,
        "roofline": roof,
        "e2e": {"value": round(wk_ops * world / (e2e_ms * 1e-3) / 1e12, 4), "unit": "TOPS", "ms_per_step": round(e2e_ms, 4),
                "h2d_bytes_per_step": int(wk.h2d_bytes), "d2h_bytes_per_step": int(wk.d2h_bytes), "steps": e2e_steps},
        "clocks": sampler.summary(),
    }
    if other:
        out["configs"] = other
    if probe:
        out["int8_mma_probe"] = probe
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, ms, cores, sample = run_oracle(name, steps=3, warmup=1, budget_s=12.0)
        out["cpu_baseline"] = {"value": round(v, 5), "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


# ---- weight gradient of a linear layer (Sec. 3.1, backward pass; G_W stays in FP32) ----------------------------------
WGRAD_SHAPE = dict(M=256, N=4096, K=4096)   # VGG16-style classifier layer 4096 -> 4096 at batch 256


def run_wgrad(args):
    """One step = one hq_linear_wgrad call (wgrad) or one hq_conv_wgrad call on the 3x3 64 -> 64 layer of cfg2 (wgrad_conv).
    Algorithmic bytes: int8 dY and X in, binary32 G_W out."""
    import torch
    from paper_2105_04246_b200 import hq
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = hq.Context(0)
    peaks, peak_kind = load_peaks()
    conv = args.workload in ("wgrad_conv", "wgrad_dw")
    g = synth.rng(4242)
    if conv:
        cs = wl.CFG2_CONV if args.workload == "wgrad_conv" else wl.CFG4_DW
        desc = hq.conv_desc(cs.N, cs.H, cs.W, cs.C, cs.K, cs.R, cs.S, cs.stride, cs.pad, cs.groups)
        dy_shape, x_shape = (cs.N, cs.Ho, cs.Wo, cs.K), (cs.N, cs.H, cs.W, cs.C)
        gw_shape = (cs.K, cs.R, cs.S) if cs.depthwise else (cs.K, cs.R, cs.S, cs.C)
        # (M, N, K) of the equivalent matrix product; depthwise: one output row, R*S*C independent sums over the pixels
        M, N, K = cs.N * cs.Ho * cs.Wo, (1 if cs.depthwise else cs.K), cs.R * cs.S * cs.C
        pool = 6 if not cs.depthwise else 2
        dy, x = synth.tiled(synth.gradients, g, dy_shape), synth.tiled(synth.relu_activations, g, x_shape)
        label = (f"{args.workload}: weight gradient of {'depthwise ' if cs.depthwise else ''}conv3x3 {cs.C}->{cs.K} @{cs.H}x{cs.W}, batch {cs.N} "
                 f"-> FP32 G_W{list(gw_shape)}")
        path = ("CUDA-core kernel on transposed words (four pixels per dot-product instruction), border sums for the zero points, conversion" if cs.depthwise else
                "dY and X packed channel-major over a padded pixel index (one copy of X per horizontal filter offset), sliced reduction on the "
                "tensor-core layer kernel (int32 slabs), slab sum + conversion")
    else:
        M, N, K = WGRAD_SHAPE["M"], WGRAD_SHAPE["N"], WGRAD_SHAPE["K"]
        dy_shape, x_shape, gw_shape = (M, N), (M, K), (N, K)
        pool = 3
        dy, x = synth.gradients(g, dy_shape), synth.relu_activations(g, x_shape)
        label = f"wgrad: weight gradient of a linear layer, dY[{M}x{N}]^T X[{M}x{K}] -> FP32 G_W[{N}x{K}]"
        path = "operand transposition, tensor-core layer kernel with binary32 epilogue"
    Ksteps, W = args.steps, max(3, args.warmup)
    dys = [torch.from_numpy(np.roll(dy.q.reshape(-1), 7919 * j).reshape(dy_shape).copy()).to(dev) for j in range(pool)]
    xs = [torch.from_numpy(np.roll(x.q.reshape(-1), 104729 * j).reshape(x_shape).copy()).to(dev) for j in range(pool)]
    gws = [torch.empty(gw_shape, dtype=torch.float32, device=dev) for _ in range(pool)]

    def call(s_, j):
        if conv:
            ctx.conv_wgrad(s_, desc, dys[j], dyq, xs[j], xq, gws[j])
        else:
            ctx.linear_wgrad(s_, M, N, K, dys[j], dyq, xs[j], xq, gws[j])
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    stream = torch.cuda.current_stream(dev)
    l0 = ctx.launch_count()
    call(stream, 0)      # also sizes the context's scratch before any capture
    launches = ctx.launch_count() - l0
    torch.cuda.synchronize()
    if args.profile:     # eager launches only, for a profiler
        for k in range(args.steps):
            call(stream, k % pool)
        torch.cuda.synchronize()
        assert ctx.get_async_error() == 0
        print(json.dumps({"profile": args.workload, "steps": args.steps, "launches_per_call": launches}))
        return
    g_full = capture(torch, call, pool)
    for _ in range(-(-W // pool)):
        g_full.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.15)
    ms_step, ms_lo, ms_hi, repeats = timed_repeats(torch, g_full.replay, pool, args.min_time, args.min_repeats)
    sampler.stop_flag = True
    sampler.join(timeout=2)
    # end to end with host buffers: both operands in from pinned memory, the gradient out to pinned memory
    h_dy, h_x = [t.cpu().pin_memory() for t in dys], [t.cpu().pin_memory() for t in xs]
    h_gw = [torch.empty(gw_shape, dtype=torch.float32).pin_memory() for _ in range(pool)]
    e2e_steps = min(Ksteps, 30)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        j = k % pool
        dys[j].copy_(h_dy[j], non_blocking=True)
        xs[j].copy_(h_x[j], non_blocking=True)
        call(stream, j)
        h_gw[j].copy_(gws[j], non_blocking=True)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    assert ctx.get_async_error() == 0
    ops = 2.0 * M * N * K
    nbytes = int(np.prod(dy_shape)) + int(np.prod(x_shape)) + 4 * int(np.prod(gw_shape))   # int8 dY and X in, binary32 G_W out
    ach = nbytes / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": round(ops / (ms_step * 1e-3) / 1e12, 3), "unit": "TOPS", "n_gpus": 1, "steps": Ksteps, "warmup": W,
        "ms_per_step": round(ms_step, 6), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "impl": "hq",
        "config": {"workload": label, "path": path,
                   "l2": f"operands and results rotate over a pool of {pool} buffer sets (> L2) inside CUDA graphs", "parallelism": "dp1"},
        "timing": {"repeats": repeats, "steps_per_repeat": pool, "ms_per_step_min": round(ms_lo, 6), "ms_per_step_max": round(ms_hi, 6),
                   "statistic": "median over repeats of one cycle through the buffer pool"},
        "gpu_launches": int(launches * pool * repeats), "launches_per_step": int(launches),
        "hbm_bytes_per_step": {"algorithmic": int(nbytes)},
        "roofline": {"bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4),
                     "kernel": ("dw_wgrad3x3_kernel + dw_wgrad_finish_kernel" if cs.depthwise else "wgrad_pack_kernel x 2 + hq_gemm_kernel (int32 slabs) + wgrad_reduce_taps_kernel") if conv else "hq_gemm_kernel (binary32 output) after transpose_rows_kernel x 2", "launch_us": round(ms_step * 1e3, 3), "traffic": None,
                     "peak_source": peak_kind, "frac_of": f"of {peak_kind}"},
        "e2e": {"value": round(ops / (e2e_ms * 1e-3) / 1e12, 4), "unit": "TOPS", "ms_per_step": round(e2e_ms, 4),
                "h2d_bytes_per_step": int(M * N + M * K), "d2h_bytes_per_step": int(4 * N * K), "steps": e2e_steps},
        "clocks": sampler.summary(),
    }
    if not args.no_cpu_baseline:
        import oracle as O
        O.build()
        t0 = time.perf_counter()
        if conv:                                      # bounded sample: the first 4 images of the batch
            nb = 4
            od = O.conv_desc(nb, cs.H, cs.W, cs.C, cs.K, cs.R, cs.S, cs.stride, cs.pad, cs.groups)
            acc = O.conv_wgrad_acc(od, dy.q[:nb], dy.zero_point, x.q[:nb], x.zero_point)
            sample_ops, sample = ops * nb / cs.N, f"the first {nb} of {cs.N} images, one call"
        else:
            Ns = N // 8                               # bounded sample: one eighth of the output rows
            acc = O.linear_wgrad_acc(dy.q[:, :Ns], dy.zero_point, x.q, x.zero_point)
            sample_ops, sample = 2.0 * M * Ns * K, f"the first {Ns} of {N} output rows, one call"
        O.scale_to_real(acc, O.acc_scale(dy.scale, x.scale))
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": round(sample_ops / dt / 1e12, 5), "unit": "TOPS", "cores": os.cpu_count() or 1, "kind": "oracle",
                               "sample": sample}
    print(json.dumps(out))


def run_profile(args):
    """Eager launches only, for a profiler.  The ranges are initialised by two dynamic steps; then, for the
    chosen layer (--layer NAME; all layers when absent), --steps in-hindsight launches rotate through the layer's buffer
    pool (more than L2, so that earlier outputs are evicted to DRAM while later launches run), then --steps dynamic ones."""
    import torch
    from paper_2105_04246_b200 import hq
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = hq.Context(0)
    if args.no_overlap:
        ctx.set_option("overlap_launches", 0)
    ctx.set_option("depthwise", args.depthwise)
    wk = GpuWorkload(args.workload, ctx, dev, seed_key=0, stochastic=args.rounding == "stochastic", pool_cap=args.pool_cap)
    stream = torch.cuda.current_stream(dev)
    names = [s.name for _, s, _ in wk.layers]
    sel = [i for i, n in enumerate(names) if args.layer in (None, n)]
    if not sel:
        raise SystemExit(f"no layer named {args.layer} in {args.workload}: {names}")
    for j in range(2):
        wk.step(stream, j, dynamic=True)
    torch.cuda.synchronize()
    for k in range(args.steps):
        wk.step(stream, k, update=False) if args.layer is None else [wk.layer_call(stream, i, k) for i in sel]
    torch.cuda.synchronize()
    if not args.no_dynamic:
        for k in range(args.steps):
            wk.step(stream, k, dynamic=True) if args.layer is None else [wk.layer_call(stream, i, k, dynamic=True) for i in sel]
        torch.cuda.synchronize()
    assert ctx.get_async_error() == 0
    print(json.dumps({"profile": args.workload, "layer": args.layer, "steps": args.steps, "pool": [wk.pool[i] for i in sel],
                      "launches": ctx.launch_count()}))


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    K, W = args.steps, max(1, min(args.warmup, 3))
    v, ms, cores, sample = run_oracle(args.workload, steps=K, warmup=W, budget_s=120.0)
    layers, _ = workload_layers(args.workload)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(v, 5), "unit": "TOPS", "n_gpus": int(os.environ.get("WORLD_SIZE", 1)),
        "steps": K, "warmup": W, "ms_per_step": round(ms, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int8", "data": "synthetic",
        "config": {"workload": f"{args.workload}: " + ", ".join(s.name for _, s, _ in layers), "path": "CPU oracle (plain loops, OpenMP over output rows)"},
        "cpu_baseline": {"value": round(v, 5), "unit": "TOPS", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(v, 5), "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="hq", choices=["hq", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg4b", "cfg5", "wgrad", "wgrad_conv", "wgrad_dw"],
                    help="cfg1..cfg5: the five layer workloads; cfg4b: backward data through cfg4's block; wgrad: the weight gradient "
                         "of a linear layer (a later row of the scope)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rounding", default="nearest", choices=["nearest", "stochastic"],
                    help="stochastic: backward-data (gradient) layers use stochastic rounding, the paper's choice for gradients")
    ap.add_argument("--depthwise", type=int, default=-1, choices=[-1, 0, 1],
                    help="depthwise layers: -1 library's choice, 0 CUDA-core kernel, 1 dense slices on the tensor cores")
    ap.add_argument("--no-overlap", action="store_true",
                    help="ordinary launches instead of programmatic stream serialization (set-up of a kernel overlapping its predecessor's tail)")
    ap.add_argument("--profile", action="store_true",
                    help="eager launches only, for a profiler: one dynamic step per pool slot (initialises the ranges), then --steps "
                         "in-hindsight launches of --layer (or whole steps), then as many dynamic ones")
    ap.add_argument("--layer", default=None, help="--profile: only this layer of the workload")
    ap.add_argument("--no-dynamic", action="store_true", help="--profile: leave the dynamic launches out")
    ap.add_argument("--pool-cap", type=int, default=MAX_POOL, help="--profile: at most this many buffer sets per layer")
    ap.add_argument("--min-time", type=float, default=0.2, help="every measurement repeats until this many seconds have been timed")
    ap.add_argument("--min-repeats", type=int, default=5, help="and at least this often; the median over the repeats is reported")
    ap.add_argument("--no-probe", action="store_true", help="skip the int8 MMA-only throughput probe")
    ap.add_argument("--probe-seconds", type=float, default=4.0, help="length of the probe's sustained run")
    ap.add_argument("--only", dest="all_configs", action="store_false",
                    help="time --workload alone; by default the per-layer rows and step values of the other four configurations are appended")
    args = ap.parse_args()
    if args.impl == "hq" and args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.profile:
        sys.exit(spawn_ranks(args))
    if args.workload in ("wgrad", "wgrad_conv", "wgrad_dw") and args.impl == "hq":
        run_wgrad(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.profile:
        run_profile(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
