"""GPU path vs CPU oracle for the rows that widen the hot path: the saturation statistic, asymmetric weights,
backward data of strided depthwise layers, prepared linear weights, and 100 free-running iterations of range tracking.
Bit-exact int8 codes, accumulators and statistics; 1e-6 relative for the binary32 range state."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2105_04246_b200 import hq, synth
from paper_2105_04246_b200.synth import QTensor
from tests.harness import GpuLayer, OracleLayer, assert_state_close
from tests.test_gpu_parity import _run_iterations, _weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hq.Context(0)
    yield c
    assert c.get_async_error() == 0
    c.close()


def _in_shape(kind, shape):
    if kind == "conv_fwd":
        return (shape["N"], shape["H"], shape["W"], shape["Cin"])
    Ho = (shape["H"] + 2 * shape.get("pad", 0) - shape.get("R", 1)) // shape.get("stride", 1) + 1
    Wo = (shape["W"] + 2 * shape.get("pad", 0) - shape.get("S", 1)) // shape.get("stride", 1) + 1
    return (shape["N"], Ho, Wo, shape["K"])


# ---- saturation statistic ---------------------------------------------------------------------------------------------
SAT_CASES = {
    "conv3x3_c64": ("conv_fwd", dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1)),
    "conv3x3_c128_k256": ("conv_fwd", dict(N=2, H=9, W=9, Cin=128, K=256, R=3, S=3, stride=1, pad=1)),
    "bwd3x3_s2": ("conv_bwd", dict(N=2, H=14, W=14, Cin=64, K=128, R=3, S=3, stride=2, pad=1)),
    "1x1_fold": ("conv_fwd", dict(N=2, H=10, W=13, Cin=24, K=144, R=1, S=1)),
    "dw3x3_c144": ("conv_fwd", dict(N=2, H=10, W=12, Cin=144, K=144, R=3, S=3, stride=1, pad=1, groups=144)),
    "dw3x3_s2": ("conv_fwd", dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32)),
    "dw_bwd_s2": ("conv_bwd", dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32)),
}


@pytest.mark.parametrize("sr_seed", [None, 1234])
@pytest.mark.parametrize("name", list(SAT_CASES))
def test_saturation_counts(ctx, name, sr_seed):
    """The input scale jumps up after the range has settled, so the previous range clips many outputs; then down again."""
    kind, shape = SAT_CASES[name]
    shape = dict(shape)
    shape.setdefault("R", 1); shape.setdefault("S", 1)
    r = synth.rng(401, len(name), shape["H"], 0 if sr_seed is None else 1)
    W = _weights(r, shape)
    mult = [1.0, 1.0, 3.0, 0.5, 6.0]

    def make_x(t):
        x = synth.signed_activations(r, _in_shape(kind, shape)) if kind == "conv_fwd" else synth.gradients(r, _in_shape(kind, shape), drift=1.0)
        x.scale *= mult[t]
        return x

    g, _ = _run_iterations(ctx, kind, W, shape, make_x, len(mult), sr_seed=sr_seed, count_sat=True)
    assert g.clipped_total > 100                         # the test saw real clipping


def test_saturation_counts_linear_and_dynamic_running(ctx):
    r = synth.rng(402)
    W = synth.uniform_int8(r, (200, 80), scale=0.003)
    g, _ = _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (130, 80), scale=0.05 * (1, 1, 4, 0.3)[t], zero_point=-7), 4,
                           count_sat=True)
    assert g.clipped_total > 100
    # running min-max on the dynamic path: the moving average lags the jump, so the dynamic path clips too
    W2 = synth.uniform_int8(r, (64, 64), scale=0.01)
    gl, ol = GpuLayer(ctx, "linear", W2, count_sat=True), O.Range()
    st = gl.state(); st["dynamic_eta"] = 0.9; gl.set_state(st)
    seen = 0
    for t, m in enumerate((1.0, 1.0, 5.0, 5.0)):
        x = synth.uniform_int8(r, (96, 64), scale=0.1 * m, zero_point=4)
        codes, _ = gl.dynamic(x)
        acc = O.linear_acc(x.q, x.zero_point, W2.q)
        s_acc = O.acc_scale(x.scale, W2.scale)
        _, want_codes = O.dynamic_running(acc, s_acc, ol, 0.9)
        assert np.array_equal(codes, want_codes)
        want = O.saturation(acc, s_acc, ol)
        got = gl.state()
        assert (int(got["last_sat_below"]), int(got["last_sat_above"])) == want, t
        seen += sum(want)
    assert seen > 100


# ---- asymmetric weights -----------------------------------------------------------------------------------------------
def _asym(w: QTensor, zw: int, r) -> QTensor:
    """The same codes read on a grid with zero point zw (any int8 bytes are valid weights)."""
    return QTensor(w.q, w.scale, zw)


ASYM_CONV = {
    "3x3_c64_k64": ("conv_fwd", dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1)),
    "3x3_c128_k256": ("conv_fwd", dict(N=2, H=9, W=9, Cin=128, K=256, R=3, S=3, stride=1, pad=1)),
    "3x3_s2": ("conv_fwd", dict(N=2, H=15, W=13, Cin=64, K=32, R=3, S=3, stride=2, pad=1)),
    "1x1_c24_fold": ("conv_fwd", dict(N=2, H=10, W=13, Cin=24, K=144, R=1, S=1)),
    "7x7_s2_c3_stem": ("conv_fwd", dict(N=2, H=30, W=26, Cin=3, K=64, R=7, S=7, stride=2, pad=3)),
    "3x3_c5_patch": ("conv_fwd", dict(N=2, H=9, W=9, Cin=5, K=24, R=3, S=3, stride=1, pad=1)),
    "bwd_3x3": ("conv_bwd", dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1)),
    "bwd_3x3_s2_odd": ("conv_bwd", dict(N=2, H=15, W=13, Cin=48, K=64, R=3, S=3, stride=2, pad=1)),
    "bwd_1x1_s2": ("conv_bwd", dict(N=2, H=14, W=14, Cin=64, K=128, R=1, S=1, stride=2, pad=0)),
    "bwd_1x1_k24_fold": ("conv_bwd", dict(N=2, H=10, W=13, Cin=144, K=24, R=1, S=1)),
    "dw3x3_c144": ("conv_fwd", dict(N=2, H=10, W=12, Cin=144, K=144, R=3, S=3, stride=1, pad=1, groups=144)),
    "dw3x3_s2_c32": ("conv_fwd", dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32)),
    "dw_bwd_c32": ("conv_bwd", dict(N=3, H=13, W=21, Cin=32, K=32, R=3, S=3, stride=1, pad=1, groups=32)),
    "dw_bwd_s2_c32": ("conv_bwd", dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32)),
}


@pytest.mark.parametrize("zw", [-128, 37])
@pytest.mark.parametrize("name", list(ASYM_CONV))
def test_asymmetric_weights_conv(ctx, name, zw):
    kind, shape = ASYM_CONV[name]
    shape = dict(shape)
    shape.setdefault("R", 1); shape.setdefault("S", 1)
    r = synth.rng(403, len(name), shape["H"], zw + 128)
    W = _asym(_weights(r, shape), zw, r)
    makers = [synth.relu_activations, synth.signed_activations, synth.image_like]
    make_x = (lambda t: makers[t % 3](r, _in_shape(kind, shape))) if kind == "conv_fwd" else (lambda t: synth.gradients(r, _in_shape(kind, shape)))
    _run_iterations(ctx, kind, W, shape, make_x, 3, sr_seed=77 if zw == 37 and kind == "conv_bwd" else None)


@pytest.mark.parametrize("M,N,K,zx,zw,use_bias", [(200, 1000, 512, -7, 127, True), (130, 24, 144, 5, -128, False), (128, 512, 1000, -3, 11, False),
                                                  (70, 40, 40, 9, -1, True), (1, 16, 16, -128, 127, False)])
def test_asymmetric_weights_linear(ctx, M, N, K, zx, zw, use_bias):
    r = synth.rng(404, M, N, K)
    W = QTensor(r.integers(-128, 128, size=(N, K), dtype=np.int8), 0.003, zw)
    bias = r.integers(-5000, 5000, size=N).astype(np.int32) if use_bias else None
    _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (M, K), scale=0.05 * (1 + 0.3 * t), zero_point=zx), 3, bias=bias, max_M=M)


# ---- prepared linear weights --------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,N,K", [(256, 128, 256), (128, 1000, 512), (128, 512, 1000), (70, 40, 40)])
def test_prepared_linear_weights(ctx, M, N, K):
    """hq_linear_prepare + hq_linear_fwd_prepared: same bytes as the oracle (and hence as hq_linear_fwd), one launch per call
    when K is a multiple of 16."""
    r = synth.rng(405, M, N, K)
    W = synth.uniform_int8(r, (N, K), scale=0.004)
    g, _ = _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (M, K), scale=0.05 * (1 + 0.3 * t), zero_point=6), 3,
                           prepared=True, max_M=M)
    x = synth.uniform_int8(r, (M, K), scale=0.05, zero_point=6)
    n0 = ctx.launch_count()
    g.hindsight(x, update=False)
    assert ctx.launch_count() - n0 == (1 if K % 16 == 0 else 2)
    if K % 16 != 0:                                       # more rows than the handle was prepared for: refused, nothing launched
        big = synth.uniform_int8(r, (M + 1, K), scale=0.05, zero_point=6)
        n1 = ctx.launch_count()
        with pytest.raises(hq.HqError) as e:
            g.hindsight(big, update=False)
        assert e.value.status == 2 and ctx.launch_count() == n1


# ---- backward data of strided depthwise layers ------------------------------------------------------------------------------
DW_BWD_STRIDED = {
    "dw3x3_s2_c32": dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32),
    "dw3x3_s2_c144_even": dict(N=2, H=12, W=14, Cin=144, K=144, R=3, S=3, stride=2, pad=1, groups=144),
    "dw5x5_s2_c48": dict(N=1, H=13, W=9, Cin=48, K=48, R=5, S=5, stride=2, pad=2, groups=48),
    "dw3x3_s3_c16_nopad": dict(N=2, H=10, W=11, Cin=16, K=16, R=3, S=3, stride=3, pad=0, groups=16),
    "dw3x3_s2_c960_7x7": dict(N=1, H=7, W=7, Cin=960, K=960, R=3, S=3, stride=2, pad=1, groups=960),
}


@pytest.mark.parametrize("sr_seed", [None, 55])
@pytest.mark.parametrize("name", list(DW_BWD_STRIDED))
def test_depthwise_bwd_data_strided(ctx, name, sr_seed):
    shape = dict(DW_BWD_STRIDED[name])
    r = synth.rng(406, len(name), shape["H"])
    W = _weights(r, shape)
    _run_iterations(ctx, "conv_bwd", W, shape, lambda t: synth.gradients(r, _in_shape("conv_bwd", shape)), 3, sr_seed=sr_seed)


# ---- 100 free-running iterations ----------------------------------------------------------------------------------------------
def _free_run(ctx, kind, W, shape, pool, iters, sr_seed=None):
    """Both sides evolve their own range state for `iters` iterations (iteration 0 dynamic, then in-hindsight) over a small
    rotating pool of inputs whose scale drifts; int8 outputs are compared at a few iterations, the state at every one."""
    r = np.random.default_rng(7)
    g = GpuLayer(ctx, kind, W, shape, sr_seed=sr_seed)
    o = OracleLayer(kind, W, shape, sr_seed=sr_seed)
    accs = [o.accumulate(x) for x in pool]                 # the integer part does not depend on the drifting scale
    drift = 1.0
    for t in range(iters):
        drift *= float(np.exp(r.normal(0.0, 0.3)))
        drift = min(max(drift, 0.05), 20.0)
        j = t % len(pool)
        x = QTensor(pool[j].q, pool[j].scale * drift, pool[j].zero_point)
        y = g.step(x)
        res = o.layer.step(accs[j], o.s_acc(x))
        if t in (0, 1, 2, 50, iters - 1):
            assert np.array_equal(y, res.q), f"iteration {t}"
        assert_state_close(g.state(), o.layer.state)
    assert int(g.state()["step"]) == iters
    return g, o


def test_hundred_iterations_cfg1(ctx):
    r = synth.rng(407)
    W = synth.uniform_int8(r, (128, 256), scale=0.01)
    pool = [synth.uniform_int8(r, (256, 256), scale=0.02) for _ in range(4)]
    _free_run(ctx, "linear", W, None, pool, 100)


SMALL_RESNET = {
    "fc": ("linear", None, (128, 512), (1000, 512)),
    "layer4.ds": ("conv_fwd", dict(N=128, H=14, W=14, Cin=256, K=512, R=1, S=1, stride=2, pad=0), None, None),
    "layer3.ds": ("conv_fwd", dict(N=128, H=28, W=28, Cin=128, K=256, R=1, S=1, stride=2, pad=0), None, None),
    "layer2.ds": ("conv_fwd", dict(N=128, H=56, W=56, Cin=64, K=128, R=1, S=1, stride=2, pad=0), None, None),
    "layer4.ds.bwd": ("conv_bwd", dict(N=128, H=14, W=14, Cin=256, K=512, R=1, S=1, stride=2, pad=0), None, None),
    "layer3.ds.bwd": ("conv_bwd", dict(N=128, H=28, W=28, Cin=128, K=256, R=1, S=1, stride=2, pad=0), None, None),
}


@pytest.mark.parametrize("name", list(SMALL_RESNET))
def test_hundred_iterations_smallest_resnet18_layers(ctx, name):
    """The six smallest layers of the ResNet-18 configuration at full batch: 100 iterations of range tracking, free running."""
    kind, shape, xs, ws = SMALL_RESNET[name]
    r = synth.rng(408, len(name))
    if kind == "linear":
        W = synth.uniform_int8(r, ws, scale=0.01)
        pool = [synth.tiled(synth.relu_activations, r, xs) for _ in range(3)]
    else:
        W = _weights(r, shape)
        make = synth.relu_activations if kind == "conv_fwd" else synth.gradients
        pool = [synth.tiled(make, r, _in_shape(kind, shape)) for _ in range(3)]
    _free_run(ctx, kind, W, shape, pool, 100, sr_seed=9 if kind == "conv_bwd" else None)
