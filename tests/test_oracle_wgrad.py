"""Pins of the oracle's linear weight gradient (Sec. 3.1, backward pass): the int32 sum over the batch of
(dy - z_dy) * (x - z_x), kept in binary32 after one multiplication by the accumulator scale."""
import numpy as np

import oracle as O


def _rand(r, shape):
    return r.integers(-128, 128, size=shape, dtype=np.int64).astype(np.int8)


def test_by_eye_one_hot_rows():
    # one sample (M = 1): the gradient is the outer product of the two corrected rows
    dy = np.array([[3, -2, 0]], np.int8)
    x = np.array([[1, 5, -4, 7]], np.int8)
    g = O.linear_wgrad_acc(dy, 1, x, -1)
    want = np.outer(np.array([2, -3, -1]), np.array([2, 6, -3, 8]))
    assert np.array_equal(g, want)
    # a sample whose gradient equals its zero point contributes nothing
    dy2 = np.vstack([dy, np.full((1, 3), 1, np.int8)])
    x2 = np.vstack([x, _rand(np.random.default_rng(1), (1, 4))])
    assert np.array_equal(O.linear_wgrad_acc(dy2, 1, x2, -1), want)


def test_against_int64_matrix_product():
    r = np.random.default_rng(7)
    for (M, N, K, zdy, zx) in [(1, 1, 1, 0, 0), (5, 3, 4, 2, -128), (37, 19, 50, -7, 11), (130, 24, 144, 127, -128)]:
        dy, x = _rand(r, (M, N)), _rand(r, (M, K))
        want = (dy.astype(np.int64) - zdy).T @ (x.astype(np.int64) - zx)
        got = O.linear_wgrad_acc(dy, zdy, x, zx)
        assert got.shape == (N, K) and np.array_equal(got.astype(np.int64), want)


def test_trace_identity_with_the_forward_layer():
    """<dY - z, (X - z_x) W^T> == <(dY - z)^T (X - z_x), W> in exact integers: the weight gradient is the adjoint of the
    forward layer with respect to the weights.  A transposed operand, a swapped zero point or a dropped sample breaks it."""
    r = np.random.default_rng(11)
    M, N, K, zdy, zx = 23, 7, 31, -5, 9
    dy, x, w = _rand(r, (M, N)), _rand(r, (M, K)), _rand(r, (N, K))
    y = O.linear_acc(x, zx, w).astype(np.int64)                      # [M][N], already pinned on its own
    lhs = int(((dy.astype(np.int64) - zdy) * y).sum())
    rhs = int((O.linear_wgrad_acc(dy, zdy, x, zx).astype(np.int64) * w.astype(np.int64)).sum())
    assert lhs == rhs


def test_real_value_is_one_binary32_multiplication():
    acc = np.array([[0, 1, -1, 3, 12345678, -16777217]], np.int32)
    s = np.float32(0.0123) * np.float32(0.5)
    got = O.scale_to_real(acc, float(s))
    want = acc.astype(np.float32) * s                               # int -> binary32 (round to nearest even), one multiplication
    assert got.dtype == np.float32 and np.array_equal(got, want)
    assert got[0, 0] == 0.0 and got[0, 1] == s and got[0, 2] == -s


# ---- convolution weight gradient ------------------------------------------------------------------
def _conv_cases():
    return [dict(N=2, H=5, W=6, C=3, K=4, R=3, S=3, stride=1, pad=1), dict(N=1, H=7, W=7, C=2, K=3, R=3, S=3, stride=2, pad=1),
            dict(N=2, H=6, W=5, C=4, K=2, R=1, S=1, stride=1, pad=0), dict(N=1, H=9, W=8, C=2, K=2, R=5, S=5, stride=2, pad=2),
            dict(N=3, H=4, W=4, C=2, K=5, R=3, S=3, stride=1, pad=0)]


def _desc(c):
    return O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], stride=c["stride"], pad=c["pad"])


def test_conv_wgrad_pointwise_is_the_linear_gradient():
    r = np.random.default_rng(21)
    c = dict(N=2, H=6, W=5, C=4, K=3, R=1, S=1, stride=1, pad=0)
    d = _desc(c)
    dy, x = _rand(r, (2, 6, 5, 3)), _rand(r, (2, 6, 5, 4))
    g = O.conv_wgrad_acc(d, dy, -3, x, 7)
    assert np.array_equal(g.reshape(3, 4), O.linear_wgrad_acc(dy.reshape(-1, 3), -3, x.reshape(-1, 4), 7))


def test_conv_wgrad_trace_identity_with_the_forward_convolution():
    """<dY - z, conv_fwd(X, W)> == <conv_wgrad(dY, X), W> in exact integers, for every geometry: ties the gradient's
    index arithmetic (strides, padding skipped, tap order) to the forward convolution, which has its own pins."""
    r = np.random.default_rng(22)
    for c in _conv_cases():
        d = _desc(c)
        Ho, Wo = O.out_hw(d)
        dy, x = _rand(r, (c["N"], Ho, Wo, c["K"])), _rand(r, (c["N"], c["H"], c["W"], c["C"]))
        w = _rand(r, (c["K"], c["R"], c["S"], c["C"]))
        zdy, zx = int(r.integers(-128, 128)), int(r.integers(-128, 128))
        y = O.conv_fwd_acc(d, x, zx, w).astype(np.int64)
        lhs = int(((dy.astype(np.int64) - zdy) * y).sum())
        rhs = int((O.conv_wgrad_acc(d, dy, zdy, x, zx).astype(np.int64) * w.astype(np.int64)).sum())
        assert lhs == rhs, c


def test_conv_wgrad_against_library_convolution():
    """torch's weight gradient of conv2d in float64 on the zero-point-corrected integers (exact below 2^53); padding
    there is zero AFTER the correction, which is the reading the oracle takes."""
    import torch
    r = np.random.default_rng(23)
    for c in _conv_cases():
        d = _desc(c)
        Ho, Wo = O.out_hw(d)
        dy, x = _rand(r, (c["N"], Ho, Wo, c["K"])), _rand(r, (c["N"], c["H"], c["W"], c["C"]))
        zdy, zx = -5, 11
        xt = torch.from_numpy((x.astype(np.float64) - zx).transpose(0, 3, 1, 2).copy())
        gt = torch.from_numpy((dy.astype(np.float64) - zdy).transpose(0, 3, 1, 2).copy())
        gw = torch.nn.grad.conv2d_weight(xt, (c["K"], c["C"], c["R"], c["S"]), gt, stride=c["stride"], padding=c["pad"])
        want = gw.numpy().transpose(0, 2, 3, 1).round().astype(np.int64)
        assert np.array_equal(O.conv_wgrad_acc(d, dy, zdy, x, zx).astype(np.int64), want), c


def test_depthwise_wgrad_trace_identity_and_library():
    """Depthwise weight gradient: adjoint of the depthwise forward convolution with respect to the filter, and torch's
    grouped conv2d weight gradient in float64."""
    import torch
    r = np.random.default_rng(24)
    for c in [dict(N=2, H=6, W=7, C=4, R=3, S=3, stride=1, pad=1), dict(N=1, H=9, W=8, C=3, R=3, S=3, stride=2, pad=1),
              dict(N=2, H=7, W=7, C=2, R=5, S=5, stride=1, pad=2)]:
        d = O.conv_desc(c["N"], c["H"], c["W"], c["C"], c["C"], c["R"], c["S"], stride=c["stride"], pad=c["pad"], groups=c["C"])
        Ho, Wo = O.out_hw(d)
        dy, x = _rand(r, (c["N"], Ho, Wo, c["C"])), _rand(r, (c["N"], c["H"], c["W"], c["C"]))
        w = _rand(r, (c["C"], c["R"], c["S"]))
        zdy, zx = 6, -9
        g = O.conv_wgrad_acc(d, dy, zdy, x, zx)
        assert g.shape == (c["C"], c["R"], c["S"])
        y = O.conv_fwd_acc(d, x, zx, w).astype(np.int64)
        assert int(((dy.astype(np.int64) - zdy) * y).sum()) == int((g.astype(np.int64) * w.astype(np.int64)).sum()), c
        xt = torch.from_numpy((x.astype(np.float64) - zx).transpose(0, 3, 1, 2).copy())
        gt = torch.from_numpy((dy.astype(np.float64) - zdy).transpose(0, 3, 1, 2).copy())
        gw = torch.nn.grad.conv2d_weight(xt, (c["C"], 1, c["R"], c["S"]), gt, stride=c["stride"], padding=c["pad"], groups=c["C"])
        assert np.array_equal(g.astype(np.int64), gw.numpy()[:, 0].round().astype(np.int64)), c
