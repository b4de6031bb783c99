"""Parity at the full sizes of the workloads, in the launch configuration the benchmark times
(default staging, whole batch, persistent grid).  The oracle evaluates these tensors in full in a
few seconds each (under a minute for the whole ResNet-18-shaped stack), so every output element is
compared, not a sample."""
import numpy as np
import pytest

import oracle as O
from paper_2105_04246_b200 import hq, synth
from paper_2105_04246_b200 import workloads as wl
from tests.harness import GpuLayer, OracleLayer, assert_state_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hq.Context(0)
    yield c
    assert c.get_async_error() == 0
    c.close()


def _shape(s):
    return dict(N=s.N, H=s.H, W=s.W, Cin=s.C, K=s.K, R=s.R, S=s.S, stride=s.stride, pad=s.pad, groups=s.groups)


def _compare(t, y, res, g, o):
    assert y.shape == res.q.shape
    bad = int((y != res.q).sum())
    assert bad == 0, f"iteration {t}: {bad} of {y.size} int8 codes differ"
    assert_state_close(g.state(), o.layer.state)


def test_cfg2_conv3x3_64_full_batch(ctx):
    s = wl.CFG2_CONV
    r = synth.rng(201)
    W = synth.weights(r, (s.K, s.R, s.S, s.C))
    g, o = GpuLayer(ctx, "conv_fwd", W, _shape(s)), OracleLayer("conv_fwd", W, _shape(s))
    for t in range(4):
        x = synth.tiled(synth.relu_activations, r, (s.N, s.H, s.W, s.C))
        x.scale *= float(np.exp(r.normal(0, 0.2)))
        if t == 0:
            acc, mn, mx, _ = g.accumulate(x)
            ref = o.accumulate(x)
            assert np.array_equal(acc, ref)
            assert (mn, mx) == O.minmax(ref)
            del acc, ref
        _compare(t, g.step(x), o.step(x), g, o)


def test_cfg3_bwd_data_256_full_batch(ctx):
    s = wl.CFG3_BWD
    r = synth.rng(202)
    W = synth.weights(r, (s.K, s.R, s.S, s.C))
    g, o = GpuLayer(ctx, "conv_bwd", W, _shape(s)), OracleLayer("conv_bwd", W, _shape(s))
    for t in range(3):
        x = synth.tiled(synth.gradients, r, (s.N, s.Ho, s.Wo, s.K))
        _compare(t, g.step(x), o.step(x), g, o)


def test_cfg3_bwd_data_256_full_batch_stochastic_rounding(ctx):
    """The gradient layer with the paper's rounding for gradients: same draws on both sides, every code equal."""
    s = wl.CFG3_BWD
    r = synth.rng(205)
    W = synth.weights(r, (s.K, s.R, s.S, s.C))
    g = GpuLayer(ctx, "conv_bwd", W, _shape(s), sr_seed=424242)
    o = OracleLayer("conv_bwd", W, _shape(s), sr_seed=424242)
    for t in range(3):
        x = synth.tiled(synth.gradients, r, (s.N, s.Ho, s.Wo, s.K))
        _compare(t, g.step(x), o.step(x), g, o)


def test_cfg4_inverted_residual_chain_full_batch(ctx):
    r = synth.rng(203)
    specs = [wl.CFG4_EXPAND, wl.CFG4_DW, wl.CFG4_PROJECT]
    Ws = [synth.weights(r, (s.K, s.R, s.S) if s.depthwise else (s.K, s.R, s.S, s.C)) for s in specs]
    gs = [GpuLayer(ctx, "conv_fwd", W, _shape(s)) for s, W in zip(specs, Ws)]
    os_ = [OracleLayer("conv_fwd", W, _shape(s)) for s, W in zip(specs, Ws)]
    s0 = specs[0]
    for t in range(2):
        xg = xo = synth.tiled(synth.signed_activations, r, (s0.N, s0.H, s0.W, s0.C))
        for g, o in zip(gs, os_):
            y, res = g.step(xg), o.step(xo)
            _compare(t, y, res, g, o)
            st = g.state()
            xg = synth.QTensor(y, float(st["scale"]), int(st["zero_point"]))          # each output feeds the next layer
            xo = synth.QTensor(res.q, o.layer.state.scale, o.layer.state.zero_point)


def test_cfg5_resnet18_stack_full_batch(ctx):
    """Every layer call of the ResNet-18-shaped workload at its full batch (the configuration the benchmark times:
    window repacking of the stem, side-by-side parity classes, padded classifier rows), dynamic initialisation and one
    in-hindsight iteration, every output element against the oracle."""
    import bench
    layers, _ = bench.workload_layers("cfg5", 1)
    r = synth.rng(204)
    for kind, s, recipe in layers:
        xsh, ysh, wsh = bench.layer_shapes(kind, s)
        if kind == "linear":
            W, shape = synth.uniform_int8(r, wsh, scale=0.01), None
        else:
            W, shape = synth.weights(r, wsh), _shape(s)
        g, o = GpuLayer(ctx, kind, W, shape), OracleLayer(kind, W, shape)
        for t in range(2):
            x = bench.make_input(recipe, r, xsh)
            x.scale *= float(np.exp(r.normal(0.0, 0.3)))
            y, res = g.step(x), o.step(x)
            assert y.shape == tuple(ysh)
            bad = int((y != res.q).sum())
            assert bad == 0, f"{s.name} iteration {t}: {bad} of {y.size} int8 codes differ"
            assert_state_close(g.state(), o.layer.state)
        del g, o
