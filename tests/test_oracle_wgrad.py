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
