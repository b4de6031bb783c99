"""Weight gradient of a linear layer on the GPU (hq_linear_wgrad) against the oracle: every binary32 value equal.
Sizes span several 128-row tiles of the transposed problem, ragged tails in all three dimensions and both zero points."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2105_04246_b200 import hq, synth
from tests.harness import Guarded

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = hq.Context(0)
    yield c
    assert c.get_async_error() == 0
    c.close()


@pytest.mark.parametrize("M,N,K", [(1, 16, 16), (7, 5, 3), (50, 130, 70), (128, 1000, 512), (300, 144, 24), (513, 40, 272), (64, 300, 1000)])
def test_linear_wgrad_matches_oracle(ctx, M, N, K):
    dev = torch.device("cuda", ctx.device)
    r = synth.rng(301, M, N, K)
    dy = synth.gradients(r, (M, N))
    x = synth.relu_activations(r, (M, K)) if (M + N) % 2 else synth.signed_activations(r, (M, K))
    dy_d, x_d = torch.from_numpy(dy.q).to(dev), torch.from_numpy(x.q).to(dev)
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    want = O.scale_to_real(O.linear_wgrad_acc(dy.q, dy.zero_point, x.q, x.zero_point), O.acc_scale(dy.scale, x.scale))
    for _ in range(2):    # the second call reuses the context's scratch with stale contents
        g_gw = Guarded((N, K), torch.float32, dev, fill=float("nan")); gw = g_gw.t
        ctx.linear_wgrad(None, M, N, K, dy_d, dyq, x_d, xq, gw)
        torch.cuda.synchronize(dev)
        g_gw.check()
        got = gw.cpu().numpy()
        bad = np.argwhere(got.view(np.uint32) != want.view(np.uint32))
        assert bad.size == 0, f"{len(bad)} mismatches, first {bad[:5]}: gpu {got[tuple(bad[0])]} oracle {want[tuple(bad[0])]}"
    assert ctx.get_async_error() == 0


def test_linear_wgrad_partial_sums_may_leave_int32(ctx):
    """70000 rows of dy - z_dy = 255 against x = 127: the sum before the zero point of x is taken out is 2.27e9 > 2^31,
    the gradient itself is 255 * 70000 * (127 - z_x).  All additions are modulo 2^32, so the result is exact."""
    dev = torch.device("cuda", ctx.device)
    M, N, K = 70000, 16, 32
    dy = np.full((M, N), 127, np.int8)
    x = np.full((M, K), 127, np.int8)
    x[:, 1] = 126
    dy_d, x_d = torch.from_numpy(dy).to(dev), torch.from_numpy(x).to(dev)
    dyq = hq.states_to_device(hq.input_state(0.5, -128), dev)
    xq = hq.states_to_device(hq.input_state(0.25, 127), dev)
    g_gw = Guarded((N, K), torch.float32, dev, fill=float("nan")); gw = g_gw.t
    ctx.linear_wgrad(None, M, N, K, dy_d, dyq, x_d, xq, gw)
    torch.cuda.synchronize(dev)
    g_gw.check()
    want = O.scale_to_real(O.linear_wgrad_acc(dy, -128, x, 127), O.acc_scale(0.5, 0.25))
    assert want[0, 0] == 0.0 and want[0, 1] == np.float32(-255 * M) * np.float32(0.125)
    assert np.array_equal(gw.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_linear_wgrad_rejections_launch_nothing(ctx):
    dev = torch.device("cuda", ctx.device)
    t = torch.zeros(1024, dtype=torch.int8, device=dev)
    st = hq.states_to_device(hq.input_state(0.1, 0), dev)
    g = torch.zeros(256, dtype=torch.float32, device=dev)
    n0 = ctx.launch_count()
    for args in [(0, 4, 4, t, st, t, st, g), (4, 4, 4, None, st, t, st, g), ((1 << 24) + 1, 4, 4, t, st, t, st, g)]:
        with pytest.raises(hq.HqError):
            ctx.linear_wgrad(None, *args)
    assert ctx.launch_count() == n0


def test_linear_wgrad_bench_size_sampled_rows(ctx):
    """The benchmark's shape (4096 -> 4096 classifier layer at batch 256): output rows sampled over the whole matrix,
    each compared in full with the oracle (the oracle computes a row block from the matching columns of dY)."""
    dev = torch.device("cuda", ctx.device)
    M, N, K = 256, 4096, 4096
    r = synth.rng(302)
    dy, x = synth.gradients(r, (M, N)), synth.relu_activations(r, (M, K))
    dy_d, x_d = torch.from_numpy(dy.q).to(dev), torch.from_numpy(x.q).to(dev)
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    gw = torch.empty((N, K), dtype=torch.float32, device=dev)
    ctx.linear_wgrad(None, M, N, K, dy_d, dyq, x_d, xq, gw)
    torch.cuda.synchronize(dev)
    got = gw.cpu().numpy()
    rows = np.unique(np.concatenate([np.arange(0, 130), np.arange(2040, 2060), np.arange(N - 70, N), r.integers(0, N, 64)]))
    want = O.scale_to_real(O.linear_wgrad_acc(np.ascontiguousarray(dy.q[:, rows]), dy.zero_point, x.q, x.zero_point),
                           O.acc_scale(dy.scale, x.scale))
    assert np.array_equal(got[rows].view(np.uint32), want.view(np.uint32))
    assert np.isfinite(got).all()


CONV_WGRAD_CASES = {
    "3x3_c64_k64": dict(N=3, H=12, W=20, Cin=64, K=64, R=3, S=3, stride=1, pad=1),
    "3x3_c16_k32_odd": dict(N=2, H=9, W=11, Cin=16, K=32, R=3, S=3, stride=1, pad=1),
    "3x3_s2_c32_k48": dict(N=2, H=15, W=13, Cin=32, K=48, R=3, S=3, stride=2, pad=1),
    "1x1_c144_k24": dict(N=2, H=10, W=13, Cin=144, K=24, R=1, S=1, stride=1, pad=0),
    "1x1_s2_c64_k128": dict(N=2, H=14, W=14, Cin=64, K=128, R=1, S=1, stride=2, pad=0),
    "5x5_c3_k20": dict(N=1, H=11, W=11, Cin=3, K=20, R=5, S=5, stride=1, pad=2),
    "3x3_c128_k256_big": dict(N=8, H=28, W=28, Cin=128, K=256, R=3, S=3, stride=1, pad=1),
    "7x7_s2_c3_k64_stem": dict(N=2, H=30, W=26, Cin=3, K=64, R=7, S=7, stride=2, pad=3),
    "3x3_nopad": dict(N=1, H=10, W=10, Cin=64, K=64, R=3, S=3, stride=1, pad=0),
    "5x5_c16_k8_pad1": dict(N=2, H=11, W=13, Cin=16, K=8, R=5, S=5, stride=1, pad=1),
    "3x3_c32_k20_wide": dict(N=2, H=6, W=70, Cin=32, K=20, R=3, S=3, stride=1, pad=1),
    "3x3_nopad_wo16": dict(N=2, H=6, W=18, Cin=16, K=16, R=3, S=3, stride=1, pad=0),
}


@pytest.mark.parametrize("windows", [-1, 1])
@pytest.mark.parametrize("name", list(CONV_WGRAD_CASES))
def test_conv_wgrad_matches_oracle(ctx, name, windows):
    """Both forms of the dense weight gradient (stride-1 layers: tensors packed over a padded pixel index; any layer: one
    transposed copy of the input per filter tap) give the oracle's bits."""
    ctx.set_option("wgrad_windows", windows)
    try:
        _conv_wgrad_case(ctx, name)
    finally:
        ctx.set_option("wgrad_windows", -1)


def _conv_wgrad_case(ctx, name):
    c = CONV_WGRAD_CASES[name]
    dev = torch.device("cuda", ctx.device)
    r = synth.rng(303, len(name), c["H"], c["Cin"])
    desc = hq.conv_desc(c["N"], c["H"], c["W"], c["Cin"], c["K"], c["R"], c["S"], stride=c["stride"], pad=c["pad"])
    od = O.conv_desc(c["N"], c["H"], c["W"], c["Cin"], c["K"], c["R"], c["S"], stride=c["stride"], pad=c["pad"])
    Ho, Wo = O.out_hw(od)
    dy = synth.gradients(r, (c["N"], Ho, Wo, c["K"]))
    x = synth.relu_activations(r, (c["N"], c["H"], c["W"], c["Cin"]))
    dy_d, x_d = torch.from_numpy(dy.q).to(dev), torch.from_numpy(x.q).to(dev)
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    want = O.scale_to_real(O.conv_wgrad_acc(od, dy.q, dy.zero_point, x.q, x.zero_point), O.acc_scale(dy.scale, x.scale))
    for _ in range(2):
        g_gw = Guarded((c["K"], c["R"], c["S"], c["Cin"]), torch.float32, dev, fill=float("nan")); gw = g_gw.t
        ctx.conv_wgrad(None, desc, dy_d, dyq, x_d, xq, gw)
        torch.cuda.synchronize(dev)
        g_gw.check()
        got = gw.cpu().numpy()
        bad = np.argwhere(got.view(np.uint32) != want.view(np.uint32))
        assert bad.size == 0, f"{len(bad)} mismatches, first {bad[:5]}: gpu {got[tuple(bad[0])]} oracle {want[tuple(bad[0])]}"
    assert ctx.get_async_error() == 0


def test_conv_wgrad_bench_size_sampled_channels(ctx):
    """The benchmark's layer (3x3, 64 -> 64, 56x56, batch 64: 200704 output pixels, 98 reduction slices): four output
    channels compared in full with the oracle, which computes them from the matching channels of dY."""
    from paper_2105_04246_b200 import workloads as wl
    cs = wl.CFG2_CONV
    dev = torch.device("cuda", ctx.device)
    r = synth.rng(304)
    dy = synth.tiled(synth.gradients, r, (cs.N, cs.Ho, cs.Wo, cs.K))
    x = synth.tiled(synth.relu_activations, r, (cs.N, cs.H, cs.W, cs.C))
    desc = hq.conv_desc(cs.N, cs.H, cs.W, cs.C, cs.K, cs.R, cs.S, cs.stride, cs.pad)
    dy_d, x_d = torch.from_numpy(dy.q).to(dev), torch.from_numpy(x.q).to(dev)
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    gw = torch.empty((cs.K, cs.R, cs.S, cs.C), dtype=torch.float32, device=dev)
    ctx.conv_wgrad(None, desc, dy_d, dyq, x_d, xq, gw)
    torch.cuda.synchronize(dev)
    got = gw.cpu().numpy()
    ks = [0, 17, 40, 63]
    od = O.conv_desc(cs.N, cs.H, cs.W, cs.C, len(ks), cs.R, cs.S, cs.stride, cs.pad)
    want = O.scale_to_real(O.conv_wgrad_acc(od, np.ascontiguousarray(dy.q[..., ks]), dy.zero_point, x.q, x.zero_point),
                           O.acc_scale(dy.scale, x.scale))
    assert np.array_equal(got[ks].view(np.uint32), want.view(np.uint32))
    assert np.isfinite(got).all() and ctx.get_async_error() == 0


DW_WGRAD_CASES = {
    "dw3x3_c144": dict(N=2, H=10, W=12, C=144, R=3, stride=1, pad=1),
    "dw3x3_s2_c32": dict(N=2, H=11, W=11, C=32, R=3, stride=2, pad=1),
    "dw3x3_c32_ragged": dict(N=3, H=13, W=21, C=32, R=3, stride=1, pad=1),
    "dw3x3_c256_nopad": dict(N=1, H=11, W=12, C=256, R=3, stride=1, pad=0),
    "dw5x5_c48": dict(N=1, H=13, W=9, C=48, R=5, stride=1, pad=2),
    "dw3x3_c320": dict(N=2, H=7, W=7, C=320, R=3, stride=1, pad=1),
    "dw3x3_c144_56": dict(N=4, H=56, W=56, C=144, R=3, stride=1, pad=1),
    "dw3x3_c64_ragged": dict(N=3, H=15, W=30, C=64, R=3, stride=1, pad=1),
    "dw3x3_c256_small": dict(N=2, H=2, W=5, C=256, R=3, stride=1, pad=1),
}


@pytest.mark.parametrize("windows", [-1, 1])
@pytest.mark.parametrize("name", list(DW_WGRAD_CASES))
def test_depthwise_wgrad_matches_oracle(ctx, name, windows):
    """Both depthwise forms (3x3 stride 1 pad 1: four pixels per dot-product instruction on transposed words with the zero
    points taken out from border sums; any other shape, and option 1: one product at a time) give the oracle's bits."""
    ctx.set_option("wgrad_windows", windows)
    try:
        _dw_wgrad_case(ctx, name)
    finally:
        ctx.set_option("wgrad_windows", -1)


def _dw_wgrad_case(ctx, name):
    c = DW_WGRAD_CASES[name]
    dev = torch.device("cuda", ctx.device)
    r = synth.rng(305, len(name), c["H"], c["C"])
    desc = hq.conv_desc(c["N"], c["H"], c["W"], c["C"], c["C"], c["R"], c["R"], stride=c["stride"], pad=c["pad"], groups=c["C"])
    od = O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["C"], c["R"], c["R"], stride=c["stride"], pad=c["pad"], groups=c["C"])
    Ho, Wo = O.out_hw(od)
    dy = synth.gradients(r, (c["N"], Ho, Wo, c["C"]))
    x = synth.relu_activations(r, (c["N"], c["H"], c["W"], c["C"]))
    dy_d, x_d = torch.from_numpy(dy.q).to(dev), torch.from_numpy(x.q).to(dev)
    dyq = hq.states_to_device(hq.input_state(dy.scale, dy.zero_point), dev)
    xq = hq.states_to_device(hq.input_state(x.scale, x.zero_point), dev)
    want = O.scale_to_real(O.conv_wgrad_acc(od, dy.q, dy.zero_point, x.q, x.zero_point), O.acc_scale(dy.scale, x.scale))
    for _ in range(2):
        g_gw = Guarded((c["C"], c["R"], c["R"]), torch.float32, dev, fill=float("nan")); gw = g_gw.t
        ctx.conv_wgrad(None, desc, dy_d, dyq, x_d, xq, gw)
        torch.cuda.synchronize(dev)
        g_gw.check()
        got = gw.cpu().numpy()
        bad = np.argwhere(got.view(np.uint32) != want.view(np.uint32))
        assert bad.size == 0, f"{len(bad)} mismatches, first {bad[:5]}: gpu {got[tuple(bad[0])]} oracle {want[tuple(bad[0])]}"
    assert ctx.get_async_error() == 0


def test_depthwise_wgrad_refuses_other_filters(ctx):
    dev = torch.device("cuda", ctx.device)
    t = torch.zeros(4096, dtype=torch.int8, device=dev)
    st = hq.states_to_device(hq.input_state(0.1, 0), dev)
    g = torch.zeros(4096, dtype=torch.float32, device=dev)
    n0 = ctx.launch_count()
    with pytest.raises(hq.HqError) as e:
        ctx.conv_wgrad(None, hq.conv_desc(1, 8, 8, 16, 16, 7, 7, stride=1, pad=3, groups=16), t, st, t, st, g)
    assert e.value.status == 2 and ctx.launch_count() == n0
