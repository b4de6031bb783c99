"""GPU path vs CPU oracle, element by element, through the C-ABI binding.

Bar: bit-exact for the int32 accumulator, its min/max, the binary32 output of the dynamic path
and every int8 code; 1e-6 relative for the binary32 running range (it is expected to be equal).
Shapes are small enough for the oracle to finish in seconds and still span several 128-row
tiles, ragged tails in M, N and K, every border class of the padding, strides and channel
counts that are not multiples of 16.
"""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2105_04246_b200 import hq, synth
from tests.harness import GpuLayer, OracleLayer, assert_state_close, oracle_range_from_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hq.Context(0)
    yield c
    assert c.get_async_error() == 0
    c.close()


def _run_iterations(ctx, kind, W, shape, make_x, iters, bias=None, eta=0.9, staging=-1, repack=-1, depthwise=-1, sr_seed=None, pair=-1,
                    count_sat=False, prepared=False, max_M=0):
    ctx.set_option("staging", staging)      # how the input reaches shared memory; results must not depend on it
    ctx.set_option("pair", pair)            # one CTA per 128-row tile or CTA pairs on 256-row tiles; likewise
    ctx.set_option("repack", repack)        # how few-channel inputs are repacked; likewise
    ctx.set_option("depthwise", depthwise)  # CUDA-core kernel or dense expansion on the tensor cores; likewise
    try:
        g = GpuLayer(ctx, kind, W, shape, bias=bias, eta=eta, sr_seed=sr_seed, count_sat=count_sat, prepared=prepared, max_M=max_M)
    finally:
        ctx.set_option("staging", -1)
        ctx.set_option("pair", -1)
        ctx.set_option("repack", -1)
        ctx.set_option("depthwise", -1)
    o = OracleLayer(kind, W, shape, bias=bias, eta=eta, sr_seed=sr_seed)
    clipped_total = 0
    for t in range(iters):
        x = make_x(t)
        before = o.layer.state.copy()
        if t == 0:
            acc, mn, mx, s_acc = g.accumulate(x)
            ref = o.accumulate(x)
            assert np.array_equal(acc, ref), f"accumulator mismatch: {np.argwhere(acc != ref)[:5]}"
            assert (mn, mx) == O.minmax(ref)
            assert s_acc == o.s_acc(x)
            yq, ws = g.dynamic(x)
            res = o.step(x)
            assert res.mode == "dynamic"
            assert np.array_equal(ws, ref.astype(np.float32) * np.float32(s_acc))
        else:
            yq, stats = g.hindsight(x)
            res = o.step(x)
            assert res.mode == "hindsight"
            assert stats[:2] == (res.mn, res.mx), (t, stats, res.mn, res.mx)
        bad = np.argwhere(yq != res.q)
        assert bad.size == 0, f"iteration {t}: {len(bad)} int8 mismatches, first {bad[:5]}, gpu {yq[tuple(bad[0])]} oracle {res.q[tuple(bad[0])]}"
        st = g.state()
        assert_state_close(st, o.layer.state)
        assert (int(st["acc_min"]), int(st["acc_max"])) == (hq.INT32_MAX, hq.INT32_MIN)   # slot emptied by the update
        assert (int(st["sat_below"]), int(st["sat_above"])) == (0, 0)
        if count_sat:
            # what the quantizer clipped: with the range that quantized this tensor (dynamic: its own; hindsight: the previous one)
            used = o.layer.state if res.mode == "dynamic" else before
            want = O.saturation(res.acc, res.s_acc, used, sr_seed, iteration=before.step)
            assert (int(st["last_sat_below"]), int(st["last_sat_above"])) == want, (t, res.mode, want)
            clipped_total += sum(want)
        else:
            assert (int(st["last_sat_below"]), int(st["last_sat_above"])) == (0, 0)
    assert ctx.get_async_error() == 0
    g.clipped_total = clipped_total
    return g, o


# ---- linear ---------------------------------------------------------------------------------
def test_cfg1_linear_ten_iterations_with_scale_drift(ctx):
    r = synth.rng(101)
    W = synth.uniform_int8(r, (128, 256), scale=0.01)
    scale = [0.02]

    def make_x(t):
        scale[0] *= float(r.uniform(0.8, 1.25))
        return synth.uniform_int8(r, (256, 256), scale=scale[0], zero_point=0)

    _run_iterations(ctx, "linear", W, None, make_x, 10)


@pytest.mark.parametrize("M,N,K,zx,use_bias", [
    (200, 1000, 512, -7, True),     # ragged M, four column tiles with a ragged last one, bias
    (130, 24, 144, 5, False),       # N below one MMA tile, K tail zero-filled
    (1, 16, 16, -128, False),       # smallest
    (515, 272, 80, 127, True),      # two column tiles of 144 (second ragged), K = 64 + 16
    (384, 8, 64, 3, False),         # N not a multiple of 16
    (128, 512, 1000, -3, False),    # K not a multiple of 16 (backward of a 512 -> 1000 classifier): padded copies
    (70, 40, 40, 9, True),
])
def test_linear_ragged(ctx, M, N, K, zx, use_bias):
    r = synth.rng(102, M, N, K)
    W = synth.uniform_int8(r, (N, K), scale=0.003)
    bias = r.integers(-5000, 5000, size=N).astype(np.int32) if use_bias else None
    _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (M, K), scale=0.05 * (1 + 0.3 * t), zero_point=zx), 3, bias=bias)


# ---- convolutions -----------------------------------------------------------------------------
FWD_CASES = {
    "3x3_c64_k64": dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1),
    "3x3_c128_k256": dict(N=2, H=9, W=9, Cin=128, K=256, R=3, S=3, stride=1, pad=1),
    "3x3_c256_k512_7x7": dict(N=5, H=7, W=7, Cin=256, K=512, R=3, S=3, stride=1, pad=1),
    "3x3_s2_c64_k128": dict(N=2, H=14, W=14, Cin=64, K=128, R=3, S=3, stride=2, pad=1),
    "3x3_s2_odd": dict(N=2, H=15, W=13, Cin=64, K=32, R=3, S=3, stride=2, pad=1),
    "1x1_s2": dict(N=2, H=14, W=14, Cin=64, K=128, R=1, S=1, stride=2, pad=0),
    "1x1_c24_k144_fold": dict(N=2, H=10, W=13, Cin=24, K=144, R=1, S=1),
    "1x1_c144_k24": dict(N=2, H=10, W=13, Cin=144, K=24, R=1, S=1),
    "1x1_c64_k32_many_tiles": dict(N=4, H=112, W=112, Cin=64, K=32, R=1, S=1),   # several tiles per CTA
    "3x3_c64_56x56": dict(N=2, H=56, W=56, Cin=64, K=64, R=3, S=3, stride=1, pad=1),
    "3x3_c128_28x28": dict(N=3, H=28, W=28, Cin=128, K=128, R=3, S=3, stride=1, pad=1),
    "3x3_c512_k512_7x7": dict(N=4, H=7, W=7, Cin=512, K=512, R=3, S=3, stride=1, pad=1),
    "7x7_c16_s1": dict(N=1, H=20, W=23, Cin=16, K=32, R=7, S=7, stride=1, pad=3),
    "5x5_c16": dict(N=1, H=11, W=11, Cin=16, K=48, R=5, S=5, stride=1, pad=2),
    "7x7_s2_c3_stem": dict(N=2, H=30, W=26, Cin=3, K=64, R=7, S=7, stride=2, pad=3),
    "3x3_c5": dict(N=2, H=9, W=9, Cin=5, K=24, R=3, S=3, stride=1, pad=1),
    "7x7_s2_c3_odd": dict(N=2, H=29, W=27, Cin=3, K=32, R=7, S=7, stride=2, pad=3),
    "5x5_s2_c4_p1": dict(N=1, H=17, W=22, Cin=4, K=16, R=5, S=5, stride=2, pad=1),
    "3x3_s4_c3": dict(N=2, H=21, W=19, Cin=3, K=16, R=3, S=3, stride=4, pad=1),
    "5x5_s3_c3": dict(N=1, H=20, W=20, Cin=3, K=16, R=5, S=5, stride=3, pad=2),
    "3x3_nopad": dict(N=1, H=10, W=10, Cin=64, K=64, R=3, S=3, stride=1, pad=0),
    # few channels with image rows a TMA box can address (W * C a multiple of 16): the fused gather kernel
    "7x7_s2_c3_w32_gather": dict(N=2, H=30, W=32, Cin=3, K=64, R=7, S=7, stride=2, pad=3),
    "7x7_s2_c3_w224_gather": dict(N=1, H=12, W=224, Cin=3, K=64, R=7, S=7, stride=2, pad=3),
    "7x7_s2_c3_w224_h16_gather": dict(N=2, H=16, W=224, Cin=3, K=64, R=7, S=7, stride=2, pad=3),
    "3x3_c3_w320_gather": dict(N=2, H=6, W=320, Cin=3, K=32, R=3, S=3, stride=1, pad=1),
    "5x5_s2_c4_w20_gather": dict(N=1, H=17, W=20, Cin=4, K=16, R=5, S=5, stride=2, pad=1),
    "3x3_c5_w16_gather": dict(N=3, H=9, W=16, Cin=5, K=48, R=3, S=3, stride=1, pad=1),
    "5x5_s3_c3_w32_gather": dict(N=2, H=20, W=32, Cin=3, K=16, R=5, S=5, stride=3, pad=2),
    "3x3_c4_w64_k256_gather": dict(N=2, H=7, W=64, Cin=4, K=256, R=3, S=3, stride=1, pad=0),
    "dw3x3_c144": dict(N=2, H=10, W=12, Cin=144, K=144, R=3, S=3, stride=1, pad=1, groups=144),
    "dw3x3_s2_c32": dict(N=2, H=11, W=11, Cin=32, K=32, R=3, S=3, stride=2, pad=1, groups=32),
    "dw3x3_c64_wide": dict(N=2, H=9, W=150, Cin=64, K=64, R=3, S=3, stride=1, pad=1, groups=64),
    "dw3x3_c32_ragged": dict(N=3, H=13, W=21, Cin=32, K=32, R=3, S=3, stride=1, pad=1, groups=32),
    "dw3x3_c256_nopad": dict(N=1, H=11, W=12, Cin=256, K=256, R=3, S=3, stride=1, pad=0, groups=256),
    "dw5x5_c48": dict(N=1, H=13, W=9, Cin=48, K=48, R=5, S=5, stride=1, pad=2, groups=48),
    "dw3x3_c320": dict(N=1, H=7, W=7, Cin=320, K=320, R=3, S=3, stride=1, pad=1, groups=320),
    "dw3x3_c192_tiles": dict(N=2, H=16, W=61, Cin=192, K=192, R=3, S=3, stride=1, pad=1, groups=192),
}


def _weights(r, shape):
    if shape.get("groups", 1) != 1:
        return synth.weights(r, (shape["K"], shape["R"], shape["S"]))
    return synth.weights(r, (shape["K"], shape["R"], shape["S"], shape["Cin"]))


@pytest.mark.parametrize("staging", [-1, 0, 1])
@pytest.mark.parametrize("name", list(FWD_CASES))
def test_conv_fwd(ctx, name, staging):
    shape = dict(FWD_CASES[name])
    shape.setdefault("R", 1); shape.setdefault("S", 1)
    r = synth.rng(103, len(name), shape["H"], shape["Cin"])
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.relu_activations, synth.signed_activations, synth.relu_activations]
    _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, staging=staging)


@pytest.mark.parametrize("depthwise", [0, 1])
@pytest.mark.parametrize("name", [n for n, c in FWD_CASES.items() if c.get("groups", 1) != 1])
def test_depthwise_both_paths(ctx, name, depthwise):
    """The CUDA-core depthwise kernel and the dense (diagonal filter) form on the tensor cores give the oracle's bytes."""
    shape = dict(FWD_CASES[name])
    r = synth.rng(105, len(name), shape["H"], depthwise)
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.relu_activations, synth.signed_activations, synth.relu_activations]
    _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, depthwise=depthwise)


@pytest.mark.parametrize("dw_staging", [0, 1, 2])
@pytest.mark.parametrize("name", ["dw3x3_c144", "dw3x3_c64_wide", "dw3x3_c32_ragged", "dw3x3_c256_nopad", "dw3x3_c192_tiles"])
def test_depthwise_cuda_core_staging(ctx, name, dw_staging):
    """CUDA-core depthwise 3x3: direct global loads, TMA-staged patches with one product per dot-product instruction, and
    TMA-staged patches transposed in registers (several tiles in both directions, ragged edges) give the oracle's bytes."""
    shape = dict(FWD_CASES[name])
    r = synth.rng(106, len(name), shape["H"], dw_staging)
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.relu_activations, synth.signed_activations, synth.relu_activations]
    ctx.set_option("depthwise_staging", dw_staging)
    try:
        _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, depthwise=0)
    finally:
        ctx.set_option("depthwise_staging", -1)


@pytest.mark.parametrize("repack", [0, 1, 2])
@pytest.mark.parametrize("name", [n for n, c in FWD_CASES.items() if c["Cin"] % 16 != 0 and c.get("R", 1) > 1])
def test_conv_fwd_few_channels_repacking(ctx, name, repack):
    """All three ways to bring few-channel inputs to the tensor cores (whole filter patches; horizontal windows per input
    row; filter windows gathered in shared memory by the fused kernel, where the shape allows) give the oracle's bytes."""
    shape = dict(FWD_CASES[name])
    r = synth.rng(104, len(name), shape["H"], repack)
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.image_like, synth.signed_activations, synth.relu_activations]
    _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, repack=repack)


@pytest.mark.parametrize("name", [n for n in FWD_CASES if n.endswith("_gather")])
def test_conv_fwd_few_channels_one_row_per_tile(ctx, name):
    """The fused few-channel kernel with tiles that stay inside one output row (the default lets them run across the ends
    of rows shorter than a tile): the same bytes."""
    shape = dict(FWD_CASES[name])
    r = synth.rng(105, len(name), shape["H"])
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.image_like, synth.signed_activations, synth.relu_activations]
    ctx.set_option("gather_span", 0)
    try:
        _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, repack=2)
    finally:
        ctx.set_option("gather_span", 1)


@pytest.mark.parametrize("producers", [1, 2])
@pytest.mark.parametrize("name", [n for n, c in FWD_CASES.items() if c.get("R", 1) == 1] + ["3x3_s2_odd", "3x3_c512_k512_7x7"])
def test_conv_fwd_operand_producers(ctx, name, producers):
    """Layers that take one input copy per filter tap, with one warp copying the input tiles or two warps copying them for
    alternate tiles (where the layer keeps its weights in shared memory; elsewhere the option changes nothing): same bytes."""
    shape = dict(FWD_CASES[name])
    r = synth.rng(106, len(name), shape["H"], producers)
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    ctx.set_option("a_producers", producers)
    try:
        _run_iterations(ctx, "conv_fwd", W, shape, lambda t: synth.relu_activations(r, in_shape), 3, staging=0)
    finally:
        ctx.set_option("a_producers", -1)


BWD_CASES = {
    "3x3_c64_k64": dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1),
    "3x3_c256_k256_14x14": dict(N=3, H=14, W=14, Cin=256, K=256, R=3, S=3, stride=1, pad=1),
    "3x3_s2_c64_k128": dict(N=2, H=14, W=14, Cin=64, K=128, R=3, S=3, stride=2, pad=1),
    "3x3_s2_odd": dict(N=2, H=15, W=13, Cin=48, K=64, R=3, S=3, stride=2, pad=1),
    "1x1_s2": dict(N=2, H=14, W=14, Cin=64, K=128, R=1, S=1, stride=2, pad=0),
    "1x1_k24_fold": dict(N=2, H=10, W=13, Cin=144, K=24, R=1, S=1),
    "1x1_k144_c24": dict(N=2, H=10, W=13, Cin=24, K=144, R=1, S=1),
}


@pytest.mark.parametrize("staging", [-1, 0, 1])
@pytest.mark.parametrize("name", list(BWD_CASES))
def test_conv_bwd_data(ctx, name, staging):
    shape = dict(BWD_CASES[name])
    r = synth.rng(104, len(name), shape["H"], shape["Cin"])
    W = _weights(r, shape)
    Ho = (shape["H"] + 2 * shape.get("pad", 0) - shape["R"]) // shape.get("stride", 1) + 1
    Wo = (shape["W"] + 2 * shape.get("pad", 0) - shape["S"]) // shape.get("stride", 1) + 1
    in_shape = (shape["N"], Ho, Wo, shape["K"])
    _run_iterations(ctx, "conv_bwd", W, shape, lambda t: synth.gradients(r, in_shape), 3, staging=staging)


# CTA pairs (tcgen05 cta_group::2): layers whose weights stream through shared memory, in both staging modes; odd image
# and tile counts leave the second CTA of the last pair with a tile of padding only
PAIR_FWD = ["3x3_c128_k256", "3x3_c256_k512_7x7", "3x3_c512_k512_7x7", "3x3_s2_c64_k128_30x30", "3x3_c256_k256_14x14_n5", "3x3_c128_k128_20x20_n3"]
PAIR_EXTRA = {
    "3x3_s2_c64_k128_30x30": dict(N=3, H=30, W=30, Cin=64, K=128, R=3, S=3, stride=2, pad=1),
    "3x3_s2_c128_k256_18x18": dict(N=3, H=18, W=18, Cin=128, K=256, R=3, S=3, stride=2, pad=1),
    "3x3_c256_k256_14x14_n5": dict(N=5, H=14, W=14, Cin=256, K=256, R=3, S=3, stride=1, pad=1),
    "3x3_c128_k128_20x20_n3": dict(N=3, H=20, W=20, Cin=128, K=320, R=3, S=3, stride=1, pad=1),
}


@pytest.mark.parametrize("cols", [0, 2, 3])
@pytest.mark.parametrize("name", ["3x3_c256_k512_7x7", "3x3_c128_k256", "3x3_c64_k64", "1x1_c144_k24"])
def test_conv_fwd_column_tiles(ctx, name, cols):
    """The split of the output channels into column tiles (option col_tiles) does not change a byte, ragged last tile included."""
    shape = dict(FWD_CASES[name])
    shape.setdefault("R", 1); shape.setdefault("S", 1)
    r = synth.rng(109, len(name), shape["H"], cols)
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.relu_activations, synth.signed_activations, synth.relu_activations]
    ctx.set_option("col_tiles", cols)
    try:
        _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3)
    finally:
        ctx.set_option("col_tiles", -1)


@pytest.mark.parametrize("staging", [0, 1])
@pytest.mark.parametrize("name", PAIR_FWD)
def test_conv_fwd_cta_pairs(ctx, name, staging):
    shape = dict(FWD_CASES.get(name) or PAIR_EXTRA[name])
    r = synth.rng(107, len(name), shape["H"], shape["Cin"])
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    makers = [synth.relu_activations, synth.signed_activations, synth.relu_activations]
    n0 = ctx.pair_launch_count()
    _run_iterations(ctx, "conv_fwd", W, shape, lambda t: makers[t % 3](r, in_shape), 3, staging=staging, pair=1)
    assert ctx.pair_launch_count() > n0, "the layer did not run as CTA pairs"


@pytest.mark.parametrize("staging", [0, 1])
@pytest.mark.parametrize("name", ["3x3_c256_k256_14x14", "3x3_s2_c128_k256_18x18"])
def test_conv_bwd_data_cta_pairs(ctx, name, staging):
    shape = dict(BWD_CASES.get(name) or PAIR_EXTRA[name])
    r = synth.rng(108, len(name), shape["H"], shape["Cin"])
    W = _weights(r, shape)
    Ho = (shape["H"] + 2 * shape.get("pad", 0) - shape["R"]) // shape.get("stride", 1) + 1
    Wo = (shape["W"] + 2 * shape.get("pad", 0) - shape["S"]) // shape.get("stride", 1) + 1
    in_shape = (shape["N"], Ho, Wo, shape["K"])
    n0 = ctx.pair_launch_count()
    _run_iterations(ctx, "conv_bwd", W, shape, lambda t: synth.gradients(r, in_shape), 3, staging=staging, pair=1)
    if staging == 0 or "s2" not in name:   # with resident input rows the small parity classes keep their weights resident: no pairs
        assert ctx.pair_launch_count() > n0, "the layer did not run as CTA pairs"


DW_BWD_CASES = {
    "dw3x3_c144": dict(N=2, H=10, W=12, Cin=144, K=144, R=3, S=3, stride=1, pad=1, groups=144),
    "dw3x3_c32_ragged": dict(N=3, H=13, W=21, Cin=32, K=32, R=3, S=3, stride=1, pad=1, groups=32),
    "dw3x3_c256_nopad": dict(N=1, H=11, W=12, Cin=256, K=256, R=3, S=3, stride=1, pad=0, groups=256),
    "dw5x5_c48": dict(N=1, H=13, W=9, Cin=48, K=48, R=5, S=5, stride=1, pad=2, groups=48),
    "dw3x3_c64_wide": dict(N=2, H=9, W=150, Cin=64, K=64, R=3, S=3, stride=1, pad=1, groups=64),
    "dw5x5_c16_pad1": dict(N=2, H=9, W=8, Cin=16, K=16, R=5, S=5, stride=1, pad=1, groups=16),
}


@pytest.mark.parametrize("dw_staging", [0, 1, 2])
@pytest.mark.parametrize("name", list(DW_BWD_CASES))
def test_depthwise_bwd_data(ctx, name, dw_staging):
    """Input gradient of a stride-1 depthwise layer (run as a forward depthwise layer over the output gradient with the
    filter turned by 180 degrees) against the oracle's backward-data definition, in both staging forms of the kernel."""
    shape = dict(DW_BWD_CASES[name])
    r = synth.rng(111, len(name), shape["H"], dw_staging)
    W = _weights(r, shape)
    Ho = shape["H"] + 2 * shape["pad"] - shape["R"] + 1
    Wo = shape["W"] + 2 * shape["pad"] - shape["S"] + 1
    in_shape = (shape["N"], Ho, Wo, shape["K"])
    ctx.set_option("depthwise_staging", dw_staging)
    try:
        _run_iterations(ctx, "conv_bwd", W, shape, lambda t: synth.gradients(r, in_shape), 3)
    finally:
        ctx.set_option("depthwise_staging", -1)


# ---- protocol and edge cases ---------------------------------------------------------------------
def test_teacher_forced_state_and_saturation(ctx):
    """The oracle is fed the GPU's own state before each step: isolates the layer kernel from the
    update kernel.  The input scale jumps up so that most codes saturate, then down."""
    r = synth.rng(105)
    shape = dict(N=2, H=8, W=8, Cin=64, K=64, R=3, S=3, stride=1, pad=1)
    W = _weights(r, shape)
    g = GpuLayer(ctx, "conv_fwd", W, shape)
    o = OracleLayer("conv_fwd", W, shape)
    mult = [1.0, 1.0, 8.0, 8.0, 0.05, 0.05]
    for t, m in enumerate(mult):
        x = synth.relu_activations(r, (2, 8, 8, 64))
        x.scale *= m
        forced = oracle_range_from_gpu(g.state())
        yq = g.step(x)
        res = o.step(x, force_state=forced)
        assert np.array_equal(yq, res.q), t
        assert_state_close(g.state(), o.layer.state)
        if t == 2:
            assert ((yq == 127) | (yq == -128)).mean() > 0.3


def test_eta_extremes_and_skipped_update(ctx):
    r = synth.rng(106)
    W = synth.uniform_int8(r, (32, 64), scale=0.01)
    for eta in (0.0, 1.0):
        _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (64, 64), scale=0.1 * (t + 1)), 4, eta=eta)
    g = GpuLayer(ctx, "linear", W)
    g.step(synth.uniform_int8(r, (64, 64), scale=0.1))
    before = g.state().copy()
    ctx.range_update(g.stream, g.yq, 1, 0.9)          # empty statistics slot: nothing may change
    torch.cuda.synchronize()
    assert g.state().tobytes() == before.tobytes()


def test_checkpoint_resume_is_identical(ctx):
    r = synth.rng(107)
    W = synth.uniform_int8(r, (48, 64), scale=0.01)
    xs = [synth.uniform_int8(r, (96, 64), scale=0.1 * (1 + t % 3)) for t in range(6)]
    a = GpuLayer(ctx, "linear", W)
    outs = [a.step(x) for x in xs]
    b = GpuLayer(ctx, "linear", W)
    for x in xs[:3]:
        b.step(x)
    saved = b.state().copy()                           # the whole state of the method is this struct
    c = GpuLayer(ctx, "linear", W)
    c.set_state(saved)
    for t in range(3, 6):
        assert np.array_equal(c.step(xs[t]), outs[t])
    assert c.state().tobytes() == a.state().tobytes()


def test_rejected_calls_launch_nothing(ctx):
    dev = torch.device("cuda", 0)
    x = torch.zeros(64 * 64 + 16, dtype=torch.int8, device=dev)
    st = hq.states_to_device(hq.new_states(2), dev)
    ws = torch.ones(1, dtype=torch.float32, device=dev)
    n0 = ctx.launch_count()
    with pytest.raises(hq.HqError) as e:
        ctx.linear_fwd(None, 64, 64, 64, x[1:], st, x, ws, None, x, st[hq.STATE_BYTES:])      # misaligned X
    assert e.value.status == 3
    with pytest.raises(hq.HqError) as e:
        ctx.linear_fwd(None, 0, 64, 64, x, st, x, ws, None, x, st[hq.STATE_BYTES:])
    assert e.value.status == 1
    with pytest.raises(hq.HqError) as e:
        ctx.linear_fwd(None, 64, 64, 64, x, None, x, ws, None, x, st[hq.STATE_BYTES:])
    assert e.value.status == 1
    with pytest.raises(hq.HqError) as e:
        ctx.weights_prepare(None, hq.conv_desc(1, 8, 8, 16, 3, 3, 3, 1, 1), hq.DIR_BWD_DATA, x)   # backward data with K = 3
    assert e.value.status == 2
    with pytest.raises(hq.HqError) as e:
        ctx.range_update(None, st, 2, 1.5)
    assert e.value.status == 1
    assert ctx.launch_count() == n0
    torch.cuda.synchronize()


# ---- two layers chained on one stream with no host synchronisation in between ----------------------
@pytest.mark.parametrize("overlap", [1, 0])
def test_chained_layers_without_host_sync(ctx, overlap):
    """Layer B consumes layer A's int8 output and A's range state directly from device memory; the calls of
    all iterations are enqueued back to back.  Checks the ordering of memory effects between consecutive
    kernels (also when a kernel's set-up is allowed to overlap its predecessor's tail) against the oracle."""
    r = synth.rng(77, overlap)
    shpA = dict(N=3, H=20, W=20, Cin=32, K=64, R=3, S=3, stride=1, pad=1)
    shpB = dict(N=3, H=20, W=20, Cin=64, K=48, R=1, S=1, stride=1, pad=0)
    WA = synth.weights(r, (64, 3, 3, 32))
    WB = synth.weights(r, (48, 1, 1, 64))
    iters = 4
    xs = [synth.signed_activations(r, (3, 20, 20, 32)) for _ in range(iters)]
    dev = torch.device("cuda", ctx.device)
    stream = torch.cuda.current_stream(dev)
    ctx.set_option("overlap_launches", overlap)
    try:
        dA, dB = hq.conv_desc(**shpA), hq.conv_desc(**shpB)
        wA = torch.from_numpy(WA.q).to(dev)
        wB = torch.from_numpy(WB.q).to(dev)
        sA = torch.tensor([WA.scale], dtype=torch.float32, device=dev)
        sB = torch.tensor([WB.scale], dtype=torch.float32, device=dev)
        pA = ctx.weights_prepare(stream, dA, hq.DIR_FWD, wA)
        pB = ctx.weights_prepare(stream, dB, hq.DIR_FWD, wB)
        states = hq.states_to_device(hq.new_states(2), dev)          # [A's output, B's output]
        nbytes = hq.RANGE_STATE_DTYPE.itemsize
        stA, stB = states[:nbytes], states[nbytes:]
        xd = [torch.from_numpy(x.q).to(dev) for x in xs]
        xq = [hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev) for x in xs]
        y1 = [torch.full((3, 20, 20, 64), 99, dtype=torch.int8, device=dev) for _ in range(iters)]
        y2 = [torch.full((3, 20, 20, 48), 99, dtype=torch.int8, device=dev) for _ in range(iters)]
        ws1 = torch.empty((3, 20, 20, 64), dtype=torch.float32, device=dev)
        ws2 = torch.empty((3, 20, 20, 48), dtype=torch.float32, device=dev)
        torch.cuda.synchronize()
        for t in range(iters):                                       # nothing below waits for the device
            if t == 0:
                ctx.dynamic_quant(stream, hq.conv_op(hq.OP_CONV_FWD, dA, xd[t], xq[t], pA, sA), ws1, y1[t], stA)
                ctx.dynamic_quant(stream, hq.conv_op(hq.OP_CONV_FWD, dB, y1[t], stA, pB, sB), ws2, y2[t], stB)
            else:
                ctx.conv_fwd(stream, dA, xd[t], xq[t], pA, sA, y1[t], stA)
                ctx.conv_fwd(stream, dB, y1[t], stA, pB, sB, y2[t], stB)
                ctx.range_update(stream, states, 2, 0.9)
        torch.cuda.synchronize()
        assert ctx.get_async_error() == 0
    finally:
        ctx.set_option("overlap_launches", 1)
    oA, oB = OracleLayer("conv_fwd", WA, shpA), OracleLayer("conv_fwd", WB, shpB)
    for t in range(iters):
        gridA = oA.layer.state.copy()                                # the range A's output is quantized with (t >= 1)
        resA = oA.step(xs[t])
        if t == 0:
            gridA = oA.layer.state.copy()                            # dynamic: the range of the tensor itself
        resB = oB.step(synth.QTensor(resA.q, gridA.scale, gridA.zero_point))
        assert np.array_equal(y1[t].cpu().numpy(), resA.q), f"layer A, iteration {t}"
        assert np.array_equal(y2[t].cpu().numpy(), resB.q), f"layer B, iteration {t}"
    got = hq.states_from_device(states)
    assert_state_close(got[0], oA.layer.state)
    assert_state_close(got[1], oB.layer.state)


# ---- stochastic rounding (the paper's rounding for gradients): same draws on both sides, bit-exact codes -----------
SR_BWD = ["3x3_c64_k64", "3x3_c256_k256_14x14", "3x3_s2_c64_k128", "3x3_s2_odd"]


@pytest.mark.parametrize("name", [n for n in SR_BWD if n in BWD_CASES])
def test_stochastic_rounding_conv_bwd_data(ctx, name):
    shape = dict(BWD_CASES[name])
    r = synth.rng(401, len(name), shape["H"])
    W = _weights(r, shape)
    Ho = (shape["H"] + 2 * shape["pad"] - shape["R"]) // shape["stride"] + 1
    Wo = (shape["W"] + 2 * shape["pad"] - shape["S"]) // shape["stride"] + 1
    in_shape = (shape["N"], Ho, Wo, shape["K"])
    g, o = _run_iterations(ctx, "conv_bwd", W, shape, lambda t: synth.gradients(r, in_shape), 4, sr_seed=20210504 + len(name))
    # the draws differ between iterations and from nearest-even: the codes of the last tensor under nearest-even
    x = synth.gradients(r, in_shape)
    acc = o.accumulate(x)
    rne = O.quantize(acc, o.s_acc(x), o.layer.state)
    sr = O.quantize_sr(acc, o.s_acc(x), o.layer.state, o.layer.sr_seed, o.layer.state.step)
    assert 0.05 < (rne != sr).mean() < 0.95
    assert np.abs(rne.astype(np.int32) - sr.astype(np.int32)).max() <= 1


@pytest.mark.parametrize("name", ["1x1_c144_k24", "3x3_c5", "3x3_c64_56x56", "dw3x3_c144", "dw3x3_s2_c32", "dw3x3_c64_wide"])
def test_stochastic_rounding_conv_fwd_shapes(ctx, name):
    """Shapes that leave the straight-line pass (ragged columns, 8-byte stores), a depthwise kernel of each kind."""
    shape = dict(FWD_CASES[name])
    shape.setdefault("R", 1); shape.setdefault("S", 1)
    r = synth.rng(402, len(name), shape["H"])
    W = _weights(r, shape)
    in_shape = (shape["N"], shape["H"], shape["W"], shape["Cin"])
    _run_iterations(ctx, "conv_fwd", W, shape, lambda t: synth.signed_activations(r, in_shape), 3, sr_seed=7 + len(name))


def test_stochastic_rounding_linear_ragged(ctx):
    r = synth.rng(403)
    W = synth.uniform_int8(r, (72, 160), scale=0.02)
    _run_iterations(ctx, "linear", W, None, lambda t: synth.uniform_int8(r, (300, 160), scale=0.05, zero_point=3), 3, sr_seed=99)


# ---- running min-max on the dynamic path (Sec. 4.1) ----------------------------------------------------------------
@pytest.mark.parametrize("eta", [0.9, 0.0])
def test_dynamic_path_running_minmax(ctx, eta):
    r = synth.rng(404, int(eta * 10))
    shape = dict(N=2, H=12, W=12, Cin=32, K=48, R=3, S=3, stride=1, pad=1)
    W = synth.weights(r, (48, 3, 3, 32))
    g = GpuLayer(ctx, "conv_fwd", W, shape)
    st = g.state().copy()
    st["dynamic_eta"] = np.float32(eta)
    g.set_state(st)
    o = OracleLayer("conv_fwd", W, shape)
    q = O.Range()
    for t in range(5):
        x = synth.signed_activations(r, (2, 12, 12, 32))
        x.scale *= float(np.exp(r.normal(0.0, 0.4)))
        y, ws = g.dynamic(x)
        acc = o.accumulate(x)
        yf, codes = O.dynamic_running(acc, o.s_acc(x), q, eta)
        assert np.array_equal(ws, yf)
        assert np.array_equal(y, codes), f"iteration {t}"
        assert_state_close(g.state(), q)
