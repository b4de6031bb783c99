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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the named layer's kernel, from the ncu captures
# summarised under profiles/ (taken with the kernels as committed; set an entry to None when its kernel changes).
# Output lines still dirty in L2 when the kernel ends are not in these counters.
NCU_TRAFFIC = {"resnet_conv3x3_64": 12992000, "resnet_conv3x3_256_bwd": 13547776, "mbv2_dw3x3": 182444800,
               "mbv2_expand": 81283328, "mbv2_project": 121651200}


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
class ClockSampler(threading.Thread):
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
                    self.samples.append([v.strip() for v in out.split(",")])
            except Exception:
                pass
            time.sleep(0.05)

    def summary(self):
        sm = [float(s[0]) for s in self.samples if s[0].replace(".", "").isdigit()]
        mx = [float(s[1]) for s in self.samples if s[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for s in self.samples for i in range(4) if len(s) >= 6 and s[2 + i].lower().startswith("active")})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None, "reasons": reasons,
                "samples": len(self.samples)}


class GpuWorkload:
    """All device buffers of one workload plus the calls of one step (hindsight or dynamic)."""

    def __init__(self, name: str, ctx, dev, pool: int, seed_key: int, stochastic: bool = False):
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
        self.state_ptr = [self.states.data_ptr() + 48 * i for i in range(n)]
        self.W, self.w_scale, self.pw, self.desc, self.x_pool, self.xq_pool, self.y_pool, self.ws = [], [], [], [], [], [], [], []
        stream = torch.cuda.current_stream(dev)
        for i, (kind, s, recipe) in enumerate(self.layers):
            xsh, ysh, wsh = layer_shapes(kind, s)
            w = synth.weights(g, wsh) if kind != "linear" else synth.uniform_int8(g, wsh, scale=0.01)
            self.W.append(torch.from_numpy(w.q).to(dev))
            self.w_scale.append(torch.tensor([w.scale], dtype=torch.float32, device=dev))
            if kind == "linear":
                self.desc.append(None)
                self.pw.append(None)
            else:
                d = hq.conv_desc(s.N, s.H, s.W, s.C, s.K, s.R, s.S, s.stride, s.pad, s.groups)
                self.desc.append(d)
                self.pw.append(ctx.weights_prepare(stream, d, hq.DIR_FWD if kind == "conv_fwd" else hq.DIR_BWD_DATA, self.W[-1]))
            if recipe is not None:
                xs, xqs = [], []
                base = make_input(recipe, g, xsh)
                for j in range(pool):
                    # pool members: the same samples rolled by a prime offset (distinct bytes at every address)
                    q = base.q if j == 0 else np.roll(base.q.reshape(-1), 104729 * j).reshape(xsh)
                    xs.append(torch.from_numpy(np.ascontiguousarray(q)).to(dev))
                    xqs.append(hq.states_to_device(hq.input_state(base.scale * (1.0 + 0.05 * (j % 3)), base.zero_point), dev))
                self.x_pool.append(xs)
                self.xq_pool.append(xqs)
            else:
                self.x_pool.append(None)
                self.xq_pool.append(None)
            self.y_pool.append([torch.empty(ysh, dtype=torch.int8, device=dev) for _ in range(pool)])
            self.ws.append(None)
        self.pool = pool
        self.ops = sum(s.ops for _, s, _ in self.layers)
        self.static_bytes = [wl.layer_static_bytes(s, kind == "conv_bwd") for kind, s, _ in self.layers]
        self.dynamic_bytes = [wl.layer_dynamic_bytes(s, kind == "conv_bwd") for kind, s, _ in self.layers]
        self.h2d_bytes = sum(int(np.prod(layer_shapes(k, s)[0])) for (k, s, r) in self.layers if r is not None)
        self.d2h_bytes = int(np.prod(layer_shapes(*self.layers[-1][:2])[1]))

    def _inputs(self, i, j):
        if self.x_pool[i] is not None:
            return self.x_pool[i][j], self.xq_pool[i][j].data_ptr()
        return self.y_pool[i - 1][j], self.state_ptr[i - 1]

    def layer_call(self, stream, i, j, dynamic=False):
        hq, ctx = self.hq, self.ctx
        kind, s, _ = self.layers[i]
        x, xq = self._inputs(i, j)
        y = self.y_pool[i][j]
        if dynamic:
            if self.ws[i] is None:
                self.ws[i] = self.torch.empty(y.shape, dtype=self.torch.float32, device=self.dev)
            if kind == "linear":
                op = hq.linear_op(s.M, s.N, s.K, x, xq, self.W[i], self.w_scale[i])
            else:
                op = hq.conv_op(hq.OP_CONV_FWD if kind == "conv_fwd" else hq.OP_CONV_BWD_DATA, self.desc[i], x, xq, self.pw[i], self.w_scale[i])
            ctx.dynamic_quant(stream, op, self.ws[i], y, self.state_ptr[i])
        elif kind == "linear":
            ctx.linear_fwd(stream, s.M, s.N, s.K, x, xq, self.W[i], self.w_scale[i], None, y, self.state_ptr[i])
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
                exchange(self.states)
            self.ctx.range_update(stream, self.states, len(self.layers), 0.9)


def capture(torch, stream_fn, reps: int):
    """Captures `reps` consecutive steps (pool member j = rep index) into one CUDA graph."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        s = torch.cuda.current_stream()
        for j in range(reps):
            stream_fn(s, j)
    return g


def time_graph(torch, graph_full, graphs_single, steps: int, pool: int, dist=None):
    """Times exactly `steps` steps: whole-pool graphs, then single-step graphs for the remainder."""
    full, rem = divmod(steps, pool)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(full):
        graph_full.replay()
    for j in range(rem):
        graphs_single[j].replay()
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    return e0.elapsed_time(e1)


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
    pool = {"cfg1": 16, "cfg2": 12, "cfg3": 12, "cfg4": 2, "cfg4b": 2, "cfg5": 2}[name]
    wk = GpuWorkload(name, ctx, dev, pool, seed_key=rank, stochastic=args.rounding == "stochastic")
    K, W = args.steps, max(3, args.warmup)
    stream = torch.cuda.current_stream(dev)
    n_layers = len(wk.layers)

    # iteration 0 of the scheme: the dynamic path initialises every range (also warms the dynamic kernels up)
    for j in range(pool):
        wk.step(stream, j, dynamic=True)
    torch.cuda.synchronize()
    l0 = ctx.launch_count()
    wk.step(stream, 0)
    launches_per_step = ctx.launch_count() - l0
    torch.cuda.synchronize()

    # graphs: the launch-bound loop is replayed from CUDA graphs (all parameters live in device memory)
    g_full = capture(torch, lambda s, j: wk.step(s, j), pool)
    g_single = [capture(torch, lambda s, _j, jj=j: wk.step(s, jj), 1) for j in range(pool)]
    g_dyn = capture(torch, lambda s, j: wk.step(s, j, dynamic=True), pool)
    g_dyn_single = [capture(torch, lambda s, _j, jj=j: wk.step(s, jj, dynamic=True), 1) for j in range(pool)]
    g_layer = [capture(torch, lambda s, j, ii=i: wk.step(s, j, only_layer=ii, update=False), pool) for i in range(n_layers)]
    g_layer_dyn = [capture(torch, lambda s, j, ii=i: wk.step(s, j, dynamic=True, only_layer=ii), pool) for i in range(n_layers)]

    for _ in range(-(-W // pool)):
        g_full.replay()
        g_dyn.replay()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.15)
    if dist is None:
        ms_total = time_graph(torch, g_full, g_single, K, pool, dist)
    else:
        # more than one rank: eager steps with the statistics all-reduce between the layers and the update
        from paper_2105_04246_b200 import parallel
        for k in range(W):
            wk.step(stream, k % pool, exchange=parallel.allreduce_stats)
        dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(K):
            wk.step(stream, k % pool, exchange=parallel.allreduce_stats)
        e1.record()
        torch.cuda.synchronize()
        dist.barrier()
        ms_total = e0.elapsed_time(e1)
    # per-layer kernel durations: the same launches replayed back to back without the update kernel
    reps = max(1, K // pool)
    layer_us, layer_dyn_us = [], []
    for i in range(n_layers):
        layer_us.append(time_graph(torch, g_layer[i], None, reps * pool, pool) * 1e3 / (reps * pool))
    ms_dyn = time_graph(torch, g_dyn, g_dyn_single, K, pool, dist)
    for i in range(n_layers):
        layer_dyn_us.append(time_graph(torch, g_layer_dyn[i], None, reps * pool, pool) * 1e3 / (reps * pool))
    sampler.stop_flag = True
    sampler.join(timeout=2)

    # end to end through the binding with host buffers: every step copies its inputs from pinned host memory, runs, and
    # copies its result back to pinned host memory.  Copies run on their own streams, ordered against the compute stream
    # with events per pool slot, so the H2D of step k+1 and the D2H of step k-1 overlap step k (as a serving loop would).
    e2e_steps = min(K, 50)
    host_in = [[x.cpu().pin_memory() for x in xs] if xs is not None else None for xs in wk.x_pool]
    host_out = [torch.empty(wk.y_pool[-1][0].shape, dtype=torch.int8).pin_memory() for _ in range(pool)]
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in range(pool)]
    ev_done = [torch.cuda.Event() for _ in range(pool)]
    ev_out = [torch.cuda.Event() for _ in range(pool)]
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        j = k % pool
        with torch.cuda.stream(s_in):
            if k >= pool:
                s_in.wait_event(ev_done[j])          # the step that last read this slot's inputs has finished
            for i in range(n_layers):
                if host_in[i] is not None:
                    wk.x_pool[i][j].copy_(host_in[i][j], non_blocking=True)
            ev_in[j].record(s_in)
        stream.wait_event(ev_in[j])
        if k >= pool:
            stream.wait_event(ev_out[j])             # the slot's previous result has left the device
        wk.step(stream, j)
        ev_done[j].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[j])
            host_out[j].copy_(wk.y_pool[-1][j], non_blocking=True)
            ev_out[j].record(s_out)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    assert ctx.get_async_error() == 0, "a device-side wait expired during the benchmark"

    if dist is not None:
        t = torch.tensor([ms_total, ms_dyn, e2e_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total, ms_dyn, e2e_ms = t.tolist()

    ms_step = ms_total / K
    tops = wk.ops * world / (ms_step * 1e-3) / 1e12
    int8_peak = peaks["bf16_tflops"] * NOMINAL_INT8_OVER_BF16
    hbm_peak = peaks["hbm_gbs"]
    per_layer = []
    for i, (kind, s, _) in enumerate(wk.layers):
        us, usd = layer_us[i], layer_dyn_us[i]
        t_tensor = s.ops / (int8_peak * 1e12) * 1e6
        t_hbm = wk.static_bytes[i] / (hbm_peak * 1e9) * 1e6
        per_layer.append({
            "layer": s.name, "kind": kind, "us": round(us, 3), "us_dynamic": round(usd, 3),
            "tops": round(s.ops / us / 1e6, 2), "gbs": round(wk.static_bytes[i] / us / 1e3, 1),
            "gbs_dynamic": round(wk.dynamic_bytes[i] / usd / 1e3, 1),
            "hbm_bytes_hindsight": int(wk.static_bytes[i]), "hbm_bytes_dynamic": int(wk.dynamic_bytes[i]),
            "bound": "alu-or-hbm" if getattr(s, "depthwise", False) else ("tensor" if t_tensor >= t_hbm else "hbm"),
            "frac_tensor": None if getattr(s, "depthwise", False) else round(t_tensor / us, 4), "frac_hbm": round(t_hbm / us, 4),
        })
    # dominant kernel of the step = the layer with the longest measured duration
    dom = max(range(n_layers), key=lambda i: layer_us[i])
    kind, s, _ = wk.layers[dom]
    t_tensor = s.ops / (int8_peak * 1e12) * 1e6
    t_hbm = wk.static_bytes[dom] / (hbm_peak * 1e9) * 1e6
    if getattr(s, "depthwise", False) or t_hbm > t_tensor:
        ach = wk.static_bytes[dom] / layer_us[dom] / 1e3
        roof = {"bound": "hbm", "achieved": round(ach, 1), "peak": hbm_peak, "unit": "GB/s", "frac": round(ach / hbm_peak, 4)}
    else:
        ach = s.ops / layer_us[dom] / 1e6
        roof = {"bound": "tensor", "achieved": round(ach, 1), "peak": round(int8_peak, 1), "unit": "TOP/s", "frac": round(ach / int8_peak, 4)}
    roof.update({"kernel": "depthwise_kernel" if getattr(s, "depthwise", False) else "hq_gemm_kernel", "layer": s.name,
                 "launch_us": round(layer_us[dom], 3), "traffic": NCU_TRAFFIC.get(s.name), "peak_source": f"{peak_kind} (int8 = bf16 burst x {NOMINAL_INT8_OVER_BF16})",
                 "frac_of": f"of {peak_kind}"})

    out = {
        "metric": METRIC, "value": round(tops, 3), "unit": "TOPS", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": round(ms_step, 6), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "impl": "hq",
        "config": {"workload": f"{name}: " + ", ".join(s.name for _, s, _ in wk.layers), "path": "in-hindsight (static requant in the epilogue + min/max)",
                   "l2": f"inputs and outputs rotate over a pool of {pool} buffer sets (> L2) inside CUDA graphs", "eta": 0.9,
                   "launch": "ordinary" if args.no_overlap else "programmatic stream serialization",
                   "rounding": "nearest even" if args.rounding == "nearest" else "stochastic for gradient layers, nearest even otherwise",
                   "parallelism": f"dp{world} (batch shards; one int32 min/max all-reduce per step before the range update)" if world > 1 else "dp1"},
        "gpu_launches": int(launches_per_step * K),
        "launches_per_step": int(launches_per_step),
        "dynamic": {"value": round(wk.ops * world / (ms_dyn / K * 1e-3) / 1e12, 3), "unit": "TOPS", "ms_per_step": round(ms_dyn / K, 6)},
        "hbm_bytes_per_step": {"hindsight": int(sum(wk.static_bytes)), "dynamic": int(sum(wk.dynamic_bytes))},
        "layers": per_layer,
        "roofline": roof,
        "e2e": {"value": round(wk.ops * world / (e2e_ms * 1e-3) / 1e12, 4), "unit": "TOPS", "ms_per_step": round(e2e_ms, 4),
                "h2d_bytes_per_step": int(wk.h2d_bytes), "d2h_bytes_per_step": int(wk.d2h_bytes), "steps": e2e_steps},
        "clocks": sampler.summary(),
    }
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
        path = ("CUDA-core kernel, integer atomics, conversion" if cs.depthwise else
                "transposed filter windows, sliced reduction on the tensor-core layer kernel (int32 slabs), slab sum + conversion")
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
    g_full = capture(torch, call, pool)
    g_single = [capture(torch, lambda s_, _j, jj=j: call(s_, jj), 1) for j in range(pool)]
    for _ in range(-(-W // pool)):
        g_full.replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.15)
    ms_total = time_graph(torch, g_full, g_single, Ksteps, pool)
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
    ms_step = ms_total / Ksteps
    ach = nbytes / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": round(ops / (ms_step * 1e-3) / 1e12, 3), "unit": "TOPS", "n_gpus": 1, "steps": Ksteps, "warmup": W,
        "ms_per_step": round(ms_step, 6), "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "impl": "hq",
        "config": {"workload": label, "path": path,
                   "l2": f"operands and results rotate over a pool of {pool} buffer sets (> L2) inside CUDA graphs", "parallelism": "dp1"},
        "gpu_launches": int(launches * Ksteps), "launches_per_step": int(launches),
        "hbm_bytes_per_step": {"algorithmic": int(nbytes)},
        "roofline": {"bound": "hbm", "achieved": round(ach, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(ach / peaks["hbm_gbs"], 4),
                     "kernel": ("dw_wgrad_kernel" if cs.depthwise else "im2col_t_kernel + hq_gemm_kernel (int32 slabs) + wgrad_reduce_kernel") if conv else "hq_gemm_kernel (binary32 output) after transpose_rows_kernel x 2", "launch_us": round(ms_step * 1e3, 3), "traffic": None,
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
    import torch
    from paper_2105_04246_b200 import hq
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    ctx = hq.Context(0)
    if args.no_overlap:
        ctx.set_option("overlap_launches", 0)
    ctx.set_option("depthwise", args.depthwise)
    wk = GpuWorkload(args.workload, ctx, dev, 2, seed_key=0, stochastic=args.rounding == "stochastic")
    stream = torch.cuda.current_stream(dev)
    for j in range(2):
        wk.step(stream, j, dynamic=True)
    torch.cuda.synchronize()
    for k in range(args.steps):
        wk.step(stream, k % 2)
    torch.cuda.synchronize()
    for k in range(args.steps):
        wk.step(stream, k % 2, dynamic=True)
    torch.cuda.synchronize()
    assert ctx.get_async_error() == 0
    print(json.dumps({"profile": args.workload, "steps": args.steps, "launches": ctx.launch_count()}))


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
    ap.add_argument("--steps", type=int, default=600)
    ap.add_argument("--warmup", type=int, default=24)
    ap.add_argument("--impl", default="hq", choices=["hq", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg4b", "cfg5", "wgrad", "wgrad_conv", "wgrad_dw"],
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
                    help="eager launches only, for a profiler: pool of 2; one dynamic step per pool member (initialises the ranges), "
                         "then --steps in-hindsight steps, then --steps dynamic steps")
    args = ap.parse_args()
    if args.workload in ("wgrad", "wgrad_conv", "wgrad_dw") and args.impl == "hq" and not args.profile:
        run_wgrad(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.profile:
        run_profile(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
