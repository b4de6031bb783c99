"""Pins for the oracle's quantizer, range update and dynamic path.

Sec. 3.2 (static vs dynamic quantization, Eq. 1), Sec. 4.1 (Eq. 2-3 and the t = 0 rule).
The paper gives no quantizer equation, so the quantizer is pinned through the properties
any 2^8-level affine quantizer with round-to-nearest must have, evaluated in float64
independently of the oracle's binary32 op sequence.
"""
import numpy as np
import pytest

import oracle as O
from paper_2105_04246_b200 import synth


def _state(q_min, q_max, step=1):
    q = O.Range(q_min=q_min, q_max=q_max, step=step)
    return O.derive(q)


RANGES = [(-1.0, 1.0), (0.0, 6.0), (0.3, 6.0), (-4.0, -0.5), (-0.013, 0.4), (-1e-6, 3e-6), (-300.0, 17.0)]


@pytest.mark.parametrize("lo,hi", RANGES)
def test_grid_invariants(lo, hi):
    q = _state(lo, hi)
    glo, ghi = min(lo, 0.0), max(hi, 0.0)                     # grid contains zero
    s = (ghi - glo) / 255.0
    assert q.scale == pytest.approx(s, rel=1e-6)
    assert q.inv_scale == pytest.approx(1.0 / s, rel=1e-6)
    assert -128 <= q.zero_point <= 127
    if lo >= 0:
        assert q.zero_point == -128                            # post-ReLU tensors use the whole grid
    if hi <= 0:
        assert q.zero_point == 127
    # the grid's ends land within half a step of the requested range
    assert abs(O.dequant(-128, q) - glo) <= 0.5 * s * (1 + 1e-5)
    assert abs(O.dequant(127, q) - ghi) <= 0.5 * s * (1 + 1e-5) + s * 1e-5
    # sweep accumulators across and beyond the range
    s_acc = float(np.float32(s / 37.0))
    a_lo, a_hi = int(glo / s_acc), int(ghi / s_acc)
    span = a_hi - a_lo
    acc = np.unique(np.linspace(a_lo - span // 2 - 5, a_hi + span // 2 + 5, 20001).astype(np.int64)).astype(np.int32)
    codes = O.quantize(acc, s_acc, q).astype(np.int64)
    assert codes.min() >= -128 and codes.max() <= 127
    assert np.all(np.diff(codes) >= 0)                         # monotone in the accumulator
    y = acc.astype(np.float64) * s_acc
    deq = float(q.scale) * (codes - q.zero_point)
    inside = (y >= O.dequant(-128, q)) & (y <= O.dequant(127, q))
    assert np.all(np.abs(deq[inside] - y[inside]) <= 0.5 * q.scale * (1 + 1e-4))
    assert np.all(codes[y < O.dequant(-128, q) - q.scale] == -128)      # saturation, not wrap-around
    assert np.all(codes[y > O.dequant(127, q) + q.scale] == 127)
    assert O.quantize(np.zeros(1, np.int32), s_acc, q)[0] == q.zero_point  # real 0 is exactly representable


def test_round_half_to_even_and_saturation():
    # scale = 1 exactly: range (-128, 127) -> s = 1, z = 0
    q = _state(-128.0, 127.0)
    assert (q.scale, q.inv_scale, q.zero_point) == (1.0, 1.0, 0)
    acc = np.array([1, 3, 5, 7, -1, -3, -5, 2, 4, 1000, -1000, 255, -257], np.int32)
    got = O.quantize(acc, 0.5, q).tolist()                     # y = acc/2: 0.5, 1.5, 2.5, 3.5, ...
    assert got == [0, 2, 2, 4, 0, -2, -2, 1, 2, 127, -128, 127, -128]
    # huge and tiny scales must not wrap
    big = np.array([2**31 - 1, -2**31], np.int32)
    assert O.quantize(big, 1e20, q).tolist() == [127, -128]


def test_degenerate_range_gives_unit_scale():
    q = _state(0.0, 0.0)
    assert (q.scale, q.inv_scale) == (1.0, 1.0)
    assert O.quantize(np.zeros(4, np.int32), 0.25, q).tolist() == [q.zero_point] * 4


def test_acc_scale_is_one_rounded_product():
    sx, sw = np.float32(0.0123), np.float32(3.9e-4)
    assert O.acc_scale(float(sx), float(sw)) == float(np.float32(sx * sw))


# ---- Eq. 2-3 -----------------------------------------------------------------------------
def test_initialisation_copies_first_minmax():
    q = O.Range()
    O.range_update(q, -50, 200, 0.5, 0.9)
    assert (q.q_min, q.q_max, q.step) == (-25.0, 100.0, 1)
    # Eq. 2-3 at t = 1 with the same tensor leave the range where it is
    O.range_update(q, -50, 200, 0.5, 0.9)
    assert q.q_min == pytest.approx(-25.0, rel=1e-6) and q.q_max == pytest.approx(100.0, rel=1e-6)


@pytest.mark.parametrize("eta", [0.9, 0.5, 0.99, 0.0, 1.0])
def test_recurrence_matches_closed_form(eta):
    g = synth.rng(20, int(eta * 100))
    T = 60
    mn = -g.integers(1, 10**6, size=T)
    mx = g.integers(1, 10**6, size=T)
    s_acc = 3.1e-4
    q = O.Range()
    e = float(np.float32(eta)); s = float(np.float32(s_acc))
    for t in range(T):
        O.range_update(q, int(mn[t]), int(mx[t]), s_acc, eta)
        # q^{t+1} = eta^t m_0 + (1-eta) sum_{j=1..t} eta^{t-j} m_j   (q^1 = q^0 = m_0)
        lo = e**t * mn[0] * s + (1 - e) * sum(e**(t - j) * mn[j] * s for j in range(1, t + 1))
        hi = e**t * mx[0] * s + (1 - e) * sum(e**(t - j) * mx[j] * s for j in range(1, t + 1))
        assert q.q_min == pytest.approx(lo, rel=2e-6)
        assert q.q_max == pytest.approx(hi, rel=2e-6)
        assert q.step == t + 1
    if eta == 0.0:
        assert q.q_min == float(np.float32(np.float32(mn[-1]) * np.float32(s_acc)))     # "previous min-max"
    if eta == 1.0:
        assert q.q_min == float(np.float32(np.float32(mn[0]) * np.float32(s_acc)))      # frozen range


def test_constant_statistics_are_a_fixed_point():
    q = O.Range()
    for _ in range(200):
        O.range_update(q, -1234, 777, 0.25, 0.9)
    assert q.q_min == pytest.approx(-308.5, rel=1e-6) and q.q_max == pytest.approx(194.25, rel=1e-6)


def test_empty_statistics_leave_state_alone():
    q = _state(-1.0, 2.0, step=3)
    before = q.astuple()
    O.range_update(q, 2**31 - 1, -2**31, 0.1, 0.9)
    assert q.astuple() == before


def test_update_moves_towards_new_statistics_with_the_right_weight():
    q = O.Range()
    O.range_update(q, -100, 100, 1.0, 0.9)
    O.range_update(q, -200, 300, 1.0, 0.9)
    assert q.q_min == pytest.approx(0.1 * -200 + 0.9 * -100, rel=1e-6)    # (1-eta) on the NEW statistic
    assert q.q_max == pytest.approx(0.1 * 300 + 0.9 * 100, rel=1e-6)


# ---- dynamic path and its relation to the static path --------------------------------------
def test_dynamic_uses_current_tensor_range():
    g = synth.rng(21)
    acc = g.integers(-90000, 50000, size=5000).astype(np.int32)
    q = O.Range()
    yf, codes = O.dynamic(acc, 1e-3, q)
    assert np.array_equal(yf, acc.astype(np.float32) * np.float32(1e-3))
    assert q.q_min == yf.min() and q.q_max == yf.max()                       # Eq. 1
    mn, mx = O.minmax(acc)
    assert q.q_min == np.float32(mn) * np.float32(1e-3) and q.q_max == np.float32(mx) * np.float32(1e-3)
    assert codes.min() == -128 and codes.max() == 127                        # the whole grid is used
    assert q.step == 1


def test_static_equals_dynamic_when_ranges_coincide():
    g = synth.rng(22)
    acc = g.integers(-4000, 9000, size=(64, 33)).astype(np.int32)
    s_acc = 7.3e-4
    layer = O.Layer(eta=0.9)
    first = layer.step(acc, s_acc)
    assert first.mode == "dynamic"
    for _ in range(6):                                                        # same tensor every iteration
        res = layer.step(acc, s_acc)
        assert res.mode == "hindsight"
        fresh = O.Range()
        _, dyn = O.dynamic(acc, s_acc, fresh)
        assert np.array_equal(res.q, dyn)
        assert layer.state.q_min == pytest.approx(fresh.q_min, rel=1e-6)
    # forcing the static path's state to the dynamic state gives identical codes for a new tensor
    acc2 = g.integers(-7000, 3000, size=(64, 33)).astype(np.int32)
    fresh = O.Range()
    _, dyn2 = O.dynamic(acc2, s_acc, fresh)
    assert np.array_equal(O.quantize(acc2, s_acc, fresh), dyn2)


def test_hindsight_uses_previous_range_not_current():
    small = np.arange(-100, 101, dtype=np.int32)
    big = small * 10
    layer = O.Layer(eta=0.9)
    layer.step(small, 1.0)
    before = layer.state.copy()
    res = layer.step(big, 1.0)
    assert np.array_equal(res.q, O.quantize(big, 1.0, before))                # quantized with the OLD range ...
    assert ((res.q == -128) | (res.q == 127)).sum() > 150                    # ... so most of it saturates
    assert layer.state.q_max == pytest.approx(0.1 * 1000 + 0.9 * 100, rel=1e-6)   # and the range then follows


# ---- running min-max (Sec. 4.1: Eq. 2-3 over the current tensor's statistics, a dynamic method) ---------------
def test_running_minmax_eta_zero_is_current_minmax():
    g = synth.rng(23)
    acc = g.integers(-7000, 3000, size=777).astype(np.int32)
    a, b = O.Range(), O.Range(q_min=-50.0, q_max=70.0, step=4)
    b = O.derive(b)
    _, cur = O.dynamic(acc, 2e-3, a)
    _, run0 = O.dynamic_running(acc, 2e-3, b, 0.0)
    assert np.array_equal(cur, run0)
    assert (a.q_min, a.q_max) == (b.q_min, b.q_max) and b.step == 5


@pytest.mark.parametrize("eta", [0.9, 0.5])
def test_running_minmax_recurrence_and_use_of_the_current_tensor(eta):
    g = synth.rng(24, int(eta * 10))
    s_acc = 1e-3
    q = O.Range()
    e = float(np.float32(eta)); s = float(np.float32(s_acc))
    lo = hi = None
    for t in range(12):
        acc = (g.integers(-9000, 9000, size=400) * (1 + t % 3)).astype(np.int32)
        mn, mx = O.minmax(acc)
        _, codes = O.dynamic_running(acc, s_acc, q, eta)
        if t == 0:
            lo, hi = mn * s, mx * s                                  # first tensor: its own min/max
        else:
            lo, hi = (1 - e) * mn * s + e * lo, (1 - e) * mx * s + e * hi   # the CURRENT tensor's statistics enter at once
        assert q.q_min == pytest.approx(lo, rel=2e-6) and q.q_max == pytest.approx(hi, rel=2e-6)
        assert q.step == t + 1
        assert np.array_equal(codes, O.quantize(acc, s_acc, q))      # quantized with the range that already contains it
    # in contrast to in-hindsight min-max, which quantizes with the range BEFORE the update
    layer = O.Layer(eta)
    layer.step(np.arange(-100, 101, dtype=np.int32), 1.0)
    before = layer.state.copy()
    big = np.arange(-1000, 1001, 10, dtype=np.int32)
    res = layer.step(big, 1.0)
    run = before.copy()
    _, run_codes = O.dynamic_running(big, 1.0, run, eta)
    assert not np.array_equal(res.q, run_codes)
    assert (run.q_min, run.q_max) == (layer.state.q_min, layer.state.q_max)    # same Eq. 2-3 numbers, used one step earlier


# ---- saturation statistic (Sec. 4: "the proportion of values that lie outside the quantization grid") ----------------
def test_saturation_counts_by_eye():
    q = O.derive(O.Range(q_min=0.0, q_max=2.55, step=1))             # 255 steps of 0.01 from 0: zero point -128
    assert q.zero_point == -128 and abs(q.scale - 0.01) < 1e-8
    s_acc = 1e-3
    #            -0.6 steps: clipped   -0.4: rounds to 0   0   2.554: level 255   2.556: level 256, clipped   far out
    acc = np.array([-6, -4, 0, 2554, 2556, 9000, -9000, 1270], np.int32)
    assert O.saturation(acc, s_acc, q) == (2, 2)
    codes = O.quantize(acc, s_acc, q)
    assert codes.tolist() == [-128, -128, -128, 127, 127, 127, -128, -1]
    assert O.saturation(np.zeros(7, np.int32), s_acc, q) == (0, 0)   # real zero is always on the grid


def test_saturation_counts_against_float64_comparison():
    g = np.random.default_rng(41)
    for lo, hi in [(-0.7, 2.3), (0.0, 5.0), (-3.0, 0.0), (-1e-3, 1e-3)]:
        q = O.derive(O.Range(q_min=lo, q_max=hi, step=1))
        s_acc = (hi - lo) / 50000.0
        acc = g.integers(-60000, 60000, size=20000).astype(np.int32)
        below, above = O.saturation(acc, s_acc, q)
        # the definition in float64: the level a value rounds to, compared with the end levels
        u = acc.astype(np.float64) * np.float64(np.float32(s_acc)) / np.float64(q.scale) + q.zero_point
        near_tie = (np.abs(u - (-128.5)) < 1e-3) | (np.abs(u - 127.5) < 1e-3)
        b64, a64 = int((np.rint(u[~near_tie]) < -128).sum()), int((np.rint(u[~near_tie]) > 127).sum())
        n_tie = int(near_tie.sum())
        assert n_tie < 20 and b64 <= below <= b64 + n_tie and a64 <= above <= a64 + n_tie
        assert below + above > 0
        # counted elements are a subset of those that carry an end code, and codes strictly inside are never counted
        codes = O.quantize(acc, s_acc, q).astype(np.int64)
        assert below <= int((codes == -128).sum()) and above <= int((codes == 127).sum())
        # the first and last level stand for themselves: a value exactly on an end level is not clipped
        s = np.float64(q.scale)
        for level, want in ((-128, (0, 0)), (127, (0, 0)), (-129, (1, 0)), (128, (0, 1))):
            on = np.array([int(np.rint((level - q.zero_point) * s / np.float64(np.float32(s_acc))))], np.int32)
            u_on = on[0] * np.float64(np.float32(s_acc)) / s + q.zero_point
            if abs(u_on - level) < 0.4:                                  # the accumulator grid is fine enough to hit the level
                assert O.saturation(on, s_acc, q) == want, (level, u_on)


def test_saturation_independent_of_order_and_additive_over_shards():
    g = np.random.default_rng(42)
    q = O.derive(O.Range(q_min=-1.0, q_max=0.5, step=3))
    acc = g.integers(-3000, 3000, size=5001).astype(np.int32)
    whole = O.saturation(acc, 1e-3, q)
    assert whole[0] > 0 and whole[1] > 0
    parts = [O.saturation(p, 1e-3, q) for p in np.array_split(g.permutation(acc), 7)]
    assert whole == (sum(p[0] for p in parts), sum(p[1] for p in parts))


def test_saturation_with_stochastic_rounding_counts_what_the_quantizer_clips():
    g = np.random.default_rng(43)
    q = O.derive(O.Range(q_min=-0.4, q_max=1.1, step=5))
    acc = g.integers(-1500, 2000, size=4000).astype(np.int32)
    s_acc, seed, it, first = 1e-3, 99, 5, 64
    below, above = O.saturation(acc, s_acc, q, sr_seed=seed, iteration=it, first=first)
    # the same draws as the (separately pinned) stochastic quantizer: floor(u + r) + z outside the levels
    y = (acc.astype(np.float32) * np.float32(s_acc)).astype(np.float32)
    u = (y * np.float32(q.inv_scale)).astype(np.float32)
    r = (np.array([O.draw16(seed, it, first + i) for i in range(acc.size)], np.float32) / np.float32(65536.0)).astype(np.float32)
    c = np.floor((u + r).astype(np.float32)).astype(np.int64) + q.zero_point
    assert (below, above) == (int((c < -128).sum()), int((c > 127).sum()))
    assert below > 0 and above > 0
    det = O.saturation(acc, s_acc, q)
    assert abs(det[0] - below) <= 0.02 * acc.size and abs(det[1] - above) <= 0.02 * acc.size   # differs only within one level of the ends
