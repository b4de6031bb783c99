"""Pins for the oracle's accumulator definitions (Sec. 3.1: MAC of 8-bit operands into
32-bit accumulators; forward output and backward input gradient).

Nothing here re-types the oracle's loops in the same form: the checks are by-eye cases,
a scatter-form brute force (the oracle gathers), the adjoint identity, and library
convolutions evaluated in float64 (exact for these magnitudes).
"""
import itertools

import numpy as np
import pytest
import torch

import oracle as O
from paper_2105_04246_b200 import synth


def _rand_i8(g, shape):
    return g.integers(-128, 128, size=shape, dtype=np.int8)


# ---- readable-by-eye cases -------------------------------------------------------------
def test_linear_identity_and_outer_product():
    g = synth.rng(1)
    X = _rand_i8(g, (5, 7))
    W = np.eye(7, dtype=np.int8)
    assert np.array_equal(O.linear_acc(X, 0, W), X.astype(np.int32))
    # K = 1 is an outer product
    x = _rand_i8(g, (6, 1)); w = _rand_i8(g, (4, 1))
    assert np.array_equal(O.linear_acc(x, 0, w), x.astype(np.int32) @ w.astype(np.int32).T)
    # zero point of the input and bias
    bias = np.arange(7, dtype=np.int32) * 1000
    ref = (X.astype(np.int64) - 3) @ W.astype(np.int64).T + bias
    assert np.array_equal(O.linear_acc(X, 3, W, bias=bias), ref)


def test_linear_is_not_transposed():
    X = np.array([[1, 2, 3]], np.int8)
    W = np.array([[1, 0, 0], [0, 0, 1]], np.int8)     # W[n][k]
    assert O.linear_acc(X, 0, W).tolist() == [[1, 3]]


def test_conv_all_ones_counts_valid_taps():
    C = 2
    d = O.conv_desc(1, 4, 4, C, 3, 3, 3, stride=1, pad=1)
    X = np.ones((1, 4, 4, C), np.int8)
    W = np.ones((3, 3, 3, C), np.int8)
    acc = O.conv_fwd_acc(d, X, 0, W)
    taps = np.array([[4, 6, 6, 4], [6, 9, 9, 6], [6, 9, 9, 6], [4, 6, 6, 4]]) * C
    for k in range(3):
        assert np.array_equal(acc[0, :, :, k], taps)
    # padding is zero in the real domain: with z_x = 1 every valid tap contributes (1-1) = 0
    assert not O.conv_fwd_acc(d, X, 1, W).any()


def test_conv_one_hot_tap_is_a_shift():
    g = synth.rng(2)
    H = W_ = 5
    X = _rand_i8(g, (2, H, W_, 3))
    for r, s in itertools.product(range(3), range(3)):
        Wt = np.zeros((3, 3, 3, 3), np.int8)
        for c in range(3):
            Wt[c, r, s, c] = 1                      # output channel c copies input channel c at tap (r,s)
        d = O.conv_desc(2, H, W_, 3, 3, 3, 3, stride=1, pad=1)
        acc = O.conv_fwd_acc(d, X, 0, Wt)
        ref = np.zeros_like(acc)
        for ho, wo in itertools.product(range(H), range(W_)):
            hi, wi = ho - 1 + r, wo - 1 + s
            if 0 <= hi < H and 0 <= wi < W_:
                ref[:, ho, wo, :] = X[:, hi, wi, :]
        assert np.array_equal(acc, ref), (r, s)


def test_depthwise_does_not_mix_channels():
    g = synth.rng(3)
    X = _rand_i8(g, (1, 6, 6, 4))
    W = _rand_i8(g, (4, 3, 3))
    d = O.conv_desc(1, 6, 6, 4, 4, 3, 3, stride=1, pad=1, groups=4)
    acc = O.conv_fwd_acc(d, X, -5, W)
    for c in range(4):
        d1 = O.conv_desc(1, 6, 6, 1, 1, 3, 3, stride=1, pad=1)
        one = O.conv_fwd_acc(d1, np.ascontiguousarray(X[..., c:c + 1]), -5, np.ascontiguousarray(W[c].reshape(1, 3, 3, 1)))
        assert np.array_equal(acc[..., c], one[..., 0])


# ---- scatter-form brute force (literal loops over every multiply) ----------------------------
CASES = [
    dict(N=1, H=4, W=4, C=2, K=3, R=3, S=3, stride=1, pad=1),
    dict(N=2, H=5, W=4, C=3, K=2, R=3, S=3, stride=2, pad=1),
    dict(N=1, H=7, W=7, C=1, K=2, R=7, S=7, stride=2, pad=3),
    dict(N=1, H=6, W=5, C=2, K=2, R=1, S=1, stride=2, pad=0),
    dict(N=1, H=5, W=5, C=2, K=2, R=3, S=3, stride=1, pad=0),
    dict(N=1, H=4, W=6, C=2, K=2, R=3, S=1, stride=(1, 2), pad=(1, 0)),
]


def _desc(c, groups=1):
    return O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], stride=c["stride"], pad=c["pad"], groups=groups)


@pytest.mark.parametrize("case", CASES)
def test_conv_fwd_and_bwd_against_scatter_loops(case):
    g = synth.rng(4, case["H"], case["R"])
    d = _desc(case)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (d.N, d.H, d.W, d.C))
    Wt = _rand_i8(g, (d.K, d.R, d.S, d.C))
    G = _rand_i8(g, (d.N, Ho, Wo, d.K))
    zx, zg = 7, -3
    y = np.zeros((d.N, Ho, Wo, d.K), np.int64)
    dx = np.zeros((d.N, d.H, d.W, d.C), np.int64)
    for n, ho, wo, k, r, s, c in itertools.product(range(d.N), range(Ho), range(Wo), range(d.K), range(d.R), range(d.S), range(d.C)):
        hi = ho * d.stride_h - d.pad_h + r
        wi = wo * d.stride_w - d.pad_w + s
        if 0 <= hi < d.H and 0 <= wi < d.W:
            w = int(Wt[k, r, s, c])
            y[n, ho, wo, k] += (int(X[n, hi, wi, c]) - zx) * w
            dx[n, hi, wi, c] += (int(G[n, ho, wo, k]) - zg) * w
    assert np.array_equal(O.conv_fwd_acc(d, X, zx, Wt), y)
    assert np.array_equal(O.conv_bwd_data_acc(d, G, zg, Wt), dx)


# ---- adjoint identity: <conv(x), g> == <x, conv^T(g)> exactly -----------------------------------
@pytest.mark.parametrize("case", CASES + [dict(N=2, H=9, W=8, C=5, K=4, R=3, S=3, stride=2, pad=1)])
@pytest.mark.parametrize("depthwise", [False, True])
def test_adjoint_identity(case, depthwise):
    g = synth.rng(5, case["H"], int(depthwise))
    c = dict(case)
    if depthwise:
        c["K"] = c["C"]
    d = _desc(c, groups=c["C"] if depthwise else 1)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (d.N, d.H, d.W, d.C))
    Wt = _rand_i8(g, (d.K, d.R, d.S) if depthwise else (d.K, d.R, d.S, d.C))
    G = _rand_i8(g, (d.N, Ho, Wo, d.K))
    lhs = int((O.conv_fwd_acc(d, X, 0, Wt).astype(np.int64) * G.astype(np.int64)).sum())
    rhs = int((X.astype(np.int64) * O.conv_bwd_data_acc(d, G, 0, Wt).astype(np.int64)).sum())
    assert lhs == rhs


# ---- library routines in float64 (exact below 2^53) -----------------------------------------
LIB_CASES = [
    dict(N=2, H=9, W=11, C=6, K=5, R=3, S=3, stride=1, pad=1),
    dict(N=2, H=12, W=10, C=4, K=8, R=3, S=3, stride=2, pad=1),
    dict(N=1, H=20, W=20, C=3, K=4, R=7, S=7, stride=2, pad=3),
    dict(N=2, H=8, W=8, C=8, K=16, R=1, S=1, stride=2, pad=0),
    dict(N=3, H=7, W=7, C=16, K=8, R=1, S=1, stride=1, pad=0),
]


@pytest.mark.parametrize("case", LIB_CASES)
@pytest.mark.parametrize("depthwise", [False, True])
def test_against_torch_float64(case, depthwise):
    g = synth.rng(6, case["H"], case["R"], int(depthwise))
    c = dict(case)
    if depthwise:
        c["K"] = c["C"]
    groups = c["C"] if depthwise else 1
    d = _desc(c, groups=groups)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (d.N, d.H, d.W, d.C))
    Wt = _rand_i8(g, (d.K, d.R, d.S) if depthwise else (d.K, d.R, d.S, d.C))
    G = _rand_i8(g, (d.N, Ho, Wo, d.K))
    zx, zg = -11, 4
    w4 = Wt.reshape(d.K, d.R, d.S, 1) if depthwise else Wt
    tw = torch.from_numpy(w4.astype(np.float64)).permute(0, 3, 1, 2).contiguous()          # [K, C/groups, R, S]
    tx = torch.from_numpy(X.astype(np.float64) - zx).permute(0, 3, 1, 2).contiguous()
    ty = torch.nn.functional.conv2d(tx, tw, stride=(d.stride_h, d.stride_w), padding=(d.pad_h, d.pad_w), groups=groups)
    assert np.array_equal(O.conv_fwd_acc(d, X, zx, Wt), ty.permute(0, 2, 3, 1).numpy().astype(np.int64))
    tg = torch.from_numpy(G.astype(np.float64) - zg).permute(0, 3, 1, 2).contiguous()
    oph = d.H - ((Ho - 1) * d.stride_h - 2 * d.pad_h + d.R)
    opw = d.W - ((Wo - 1) * d.stride_w - 2 * d.pad_w + d.S)
    tdx = torch.nn.functional.conv_transpose2d(tg, tw, stride=(d.stride_h, d.stride_w), padding=(d.pad_h, d.pad_w),
                                               output_padding=(oph, opw), groups=groups)
    assert np.array_equal(O.conv_bwd_data_acc(d, G, zg, Wt), tdx.permute(0, 2, 3, 1).numpy().astype(np.int64))


def test_linear_against_numpy_int64():
    g = synth.rng(7)
    X = _rand_i8(g, (33, 70)); W = _rand_i8(g, (19, 70))
    bias = g.integers(-10**6, 10**6, size=19).astype(np.int32)
    ref = (X.astype(np.int64) + 128) @ W.astype(np.int64).T + bias
    assert np.array_equal(O.linear_acc(X, -128, W, bias=bias), ref)


# ---- sampled evaluation equals the full tensor -----------------------------------------
def test_point_evaluation_matches_full_tensor():
    g = synth.rng(8)
    d = O.conv_desc(2, 9, 8, 5, 4, 3, 3, stride=2, pad=1)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (2, 9, 8, 5)); Wt = _rand_i8(g, (4, 3, 3, 5)); G = _rand_i8(g, (2, Ho, Wo, 4))
    full = O.conv_fwd_acc(d, X, 9, Wt).ravel()
    idx = g.integers(0, full.size, size=50)
    assert np.array_equal(O.conv_fwd_acc_at(d, X, 9, Wt, idx), full[idx])
    fullb = O.conv_bwd_data_acc(d, G, -2, Wt).ravel()
    idx = g.integers(0, fullb.size, size=50)
    assert np.array_equal(O.conv_bwd_data_acc_at(d, G, -2, Wt, idx), fullb[idx])
    Xl = _rand_i8(g, (10, 12)); Wl = _rand_i8(g, (6, 12))
    fl = O.linear_acc(Xl, 1, Wl).ravel()
    idx = np.arange(60)
    assert np.array_equal(O.linear_acc_at(Xl, 1, Wl, idx), fl)


def test_statistics_are_exact_extremes_in_any_order():
    g = synth.rng(9)
    acc = g.integers(-2**31, 2**31, size=10007, dtype=np.int64).astype(np.int32)
    assert O.minmax(acc) == (int(acc.min()), int(acc.max()))
    perm = g.permutation(acc.size)
    assert O.minmax(acc[perm]) == (int(acc.min()), int(acc.max()))
    # reducing tile by tile in a shuffled order gives the same pair
    tiles = np.array_split(acc[perm], 37)
    lo = min(O.minmax(t)[0] for t in tiles); hi = max(O.minmax(t)[1] for t in tiles)
    assert (lo, hi) == (int(acc.min()), int(acc.max()))
    assert O.minmax(np.array([5], np.int32)) == (5, 5)


# ---- weight zero point (asymmetric weights: every loop takes z_w) ------------------------------------
def test_weight_zero_point_by_eye():
    # weights that all equal their zero point are real zeros: nothing accumulates, whatever the input
    g = synth.rng(10)
    X = _rand_i8(g, (3, 8))
    assert not O.linear_acc(X, 5, np.full((4, 8), -7, np.int8), zw=-7).any()
    d = O.conv_desc(1, 5, 5, 2, 3, 3, 3, stride=1, pad=1)
    Xc = _rand_i8(g, (1, 5, 5, 2))
    assert not O.conv_fwd_acc(d, Xc, 3, np.full((3, 3, 3, 2), 9, np.int8), zw=9).any()
    assert not O.conv_bwd_data_acc(d, Xc[..., :1].repeat(3, -1), 3, np.full((3, 3, 3, 2), 9, np.int8), zw=9).any()
    # all-ones input, weights one above their zero point: the count of valid taps (padding contributes nothing)
    acc = O.conv_fwd_acc(d, np.ones((1, 5, 5, 2), np.int8), 0, np.full((3, 3, 3, 2), 10, np.int8), zw=9)
    taps = np.array([[4, 6, 6, 6, 4], [6, 9, 9, 9, 6], [6, 9, 9, 9, 6], [6, 9, 9, 9, 6], [4, 6, 6, 6, 4]]) * 2
    assert np.array_equal(acc[0, :, :, 0], taps)
    # a single row, readable: (1-1, 2-1, 3-1) . (4+2, 0+2, -2+2) = 0*6 + 1*2 + 2*0
    assert O.linear_acc(np.array([[1, 2, 3]], np.int8), 1, np.array([[4, 0, -2]], np.int8), zw=-2).tolist() == [[2]]


def test_linear_weight_zero_point_against_numpy_int64():
    g = synth.rng(11)
    X = _rand_i8(g, (21, 50)); W = _rand_i8(g, (13, 50))
    bias = g.integers(-10**5, 10**5, size=13).astype(np.int32)
    for zx, zw in [(-128, 127), (17, -128), (0, 5)]:
        ref = (X.astype(np.int64) - zx) @ (W.astype(np.int64) - zw).T + bias
        assert np.array_equal(O.linear_acc(X, zx, W, zw=zw, bias=bias), ref)
        idx = g.integers(0, ref.size, size=40)
        assert np.array_equal(O.linear_acc_at(X, zx, W, idx, zw=zw, bias=bias), ref.ravel()[idx])


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("zw", [-128, 6, 127])
def test_conv_weight_zero_point_against_scatter_loops(case, zw):
    g = synth.rng(12, case["H"], case["R"], zw + 128)
    d = _desc(case)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (d.N, d.H, d.W, d.C))
    Wt = _rand_i8(g, (d.K, d.R, d.S, d.C))
    G = _rand_i8(g, (d.N, Ho, Wo, d.K))
    zx, zg = -9, 12
    y = np.zeros((d.N, Ho, Wo, d.K), np.int64)
    dx = np.zeros((d.N, d.H, d.W, d.C), np.int64)
    for n, ho, wo, k, r, s, c in itertools.product(range(d.N), range(Ho), range(Wo), range(d.K), range(d.R), range(d.S), range(d.C)):
        hi = ho * d.stride_h - d.pad_h + r
        wi = wo * d.stride_w - d.pad_w + s
        if 0 <= hi < d.H and 0 <= wi < d.W:
            w = int(Wt[k, r, s, c]) - zw
            y[n, ho, wo, k] += (int(X[n, hi, wi, c]) - zx) * w
            dx[n, hi, wi, c] += (int(G[n, ho, wo, k]) - zg) * w
    assert np.array_equal(O.conv_fwd_acc(d, X, zx, Wt, zw), y)
    assert np.array_equal(O.conv_bwd_data_acc(d, G, zg, Wt, zw), dx)
    idx = g.integers(0, y.size, size=min(30, y.size))
    assert np.array_equal(O.conv_fwd_acc_at(d, X, zx, Wt, idx, zw), y.ravel()[idx])
    idx = g.integers(0, dx.size, size=min(30, dx.size))
    assert np.array_equal(O.conv_bwd_data_acc_at(d, G, zg, Wt, idx, zw), dx.ravel()[idx])


@pytest.mark.parametrize("case", LIB_CASES[:3])
@pytest.mark.parametrize("depthwise", [False, True])
def test_weight_zero_point_against_torch_float64(case, depthwise):
    g = synth.rng(13, case["H"], case["R"], int(depthwise))
    c = dict(case)
    if depthwise:
        c["K"] = c["C"]
    groups = c["C"] if depthwise else 1
    d = _desc(c, groups=groups)
    Ho, Wo = O.out_hw(d)
    X = _rand_i8(g, (d.N, d.H, d.W, d.C))
    Wt = _rand_i8(g, (d.K, d.R, d.S) if depthwise else (d.K, d.R, d.S, d.C))
    G = _rand_i8(g, (d.N, Ho, Wo, d.K))
    zx, zg, zw = 23, -6, -31
    w4 = Wt.reshape(d.K, d.R, d.S, 1) if depthwise else Wt
    tw = torch.from_numpy(w4.astype(np.float64) - zw).permute(0, 3, 1, 2).contiguous()
    tx = torch.from_numpy(X.astype(np.float64) - zx).permute(0, 3, 1, 2).contiguous()
    ty = torch.nn.functional.conv2d(tx, tw, stride=(d.stride_h, d.stride_w), padding=(d.pad_h, d.pad_w), groups=groups)
    assert np.array_equal(O.conv_fwd_acc(d, X, zx, Wt, zw), ty.permute(0, 2, 3, 1).numpy().astype(np.int64))
    tg = torch.from_numpy(G.astype(np.float64) - zg).permute(0, 3, 1, 2).contiguous()
    oph = d.H - ((Ho - 1) * d.stride_h - 2 * d.pad_h + d.R)
    opw = d.W - ((Wo - 1) * d.stride_w - 2 * d.pad_w + d.S)
    tdx = torch.nn.functional.conv_transpose2d(tg, tw, stride=(d.stride_h, d.stride_w), padding=(d.pad_h, d.pad_w),
                                               output_padding=(oph, opw), groups=groups)
    assert np.array_equal(O.conv_bwd_data_acc(d, G, zg, Wt, zw), tdx.permute(0, 2, 3, 1).numpy().astype(np.int64))
