"""Pins for the oracle's stochastic rounding (the paper quantizes gradients with stochastic rounding and
prints no formula for it; the conventions are the oracle's readings R-18..R-20).

The generator is pinned to the known-answer vectors published with it; the rounding is pinned through what
any stochastic rounding must satisfy, evaluated independently of the oracle's binary32 op sequence."""
import os

import numpy as np
import pytest

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def _state(lo, hi, step=1):
    return O.derive(O.Range(q_min=lo, q_max=hi, step=step))


def test_philox_known_answers():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row]
        assert O.philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_draw_layout_and_reproducibility():
    seed, it = 1234, 7
    for block in (0, 1, 5, (1 << 32) + 3):                       # the block index spans two counter words
        w = O.philox4x32_10([block & 0xFFFFFFFF, block >> 32, it, 0], [seed, 0])
        halves = []
        for word in w:
            halves += [word & 0xFFFF, word >> 16]
        got = [O.draw16(seed, it, 8 * block + k) for k in range(8)]
        assert got == halves
    assert O.draw16(seed, it, 42) == O.draw16(seed, it, 42)
    a = [O.draw16(seed, it, e) for e in range(64)]
    assert a != [O.draw16(seed, it + 1, e) for e in range(64)]  # a new iteration draws anew
    assert a != [O.draw16(seed + 1, it, e) for e in range(64)]


def test_result_is_a_neighbour_of_u_and_exact_on_integers():
    q = _state(-128.0, 127.0)                                    # scale 1, zero point 0
    assert (q.scale, q.zero_point) == (1.0, 0)
    acc = np.arange(-300, 301, dtype=np.int32)
    for s_acc in (0.25, 0.5, 1.0):
        got = O.quantize_sr(acc, s_acc, q, seed=5, iteration=3).astype(np.int64)
        u = acc.astype(np.float64) * s_acc
        lo, hi = np.clip(np.floor(u), -128, 127), np.clip(np.ceil(u), -128, 127)
        assert np.all((got == lo) | (got == hi))
        integer = u == np.floor(u)
        assert np.array_equal(got[integer], np.clip(u[integer], -128, 127).astype(np.int64))   # r < 1 never carries


def test_matches_the_definition_evaluated_in_float64():
    g = np.random.default_rng(31)
    q = _state(-3.7, 9.1)
    acc = g.integers(-60000, 120000, size=4096).astype(np.int32)
    s_acc = 1.1e-4
    got = O.quantize_sr(acc, s_acc, q, seed=99, iteration=12, first=1000).astype(np.int64)
    y = (acc.astype(np.float32) * np.float32(s_acc)).astype(np.float32)
    u = (y * np.float32(q.inv_scale)).astype(np.float64)
    r = np.array([O.draw16(99, 12, 1000 + i) for i in range(acc.size)], np.float64) / 65536.0
    t = u + r                                                    # exact sum; the oracle rounds it to binary32 once
    exp = np.clip(np.floor(t) + q.zero_point, -128, 127).astype(np.int64)
    near_integer = np.abs(t - np.rint(t)) < 1e-4                 # only there may the binary32 rounding of u + r decide
    assert np.array_equal(got[~near_integer], exp[~near_integer])
    assert np.all(np.abs(got[near_integer] - exp[near_integer]) <= 1)
    assert near_integer.mean() < 0.01


def test_unbiased_over_draws():
    q = _state(-128.0, 127.0)
    fracs = np.array([0.0, 0.1, 0.25, 0.5, 0.77, 0.999], np.float64)
    n = 40000
    for f in fracs:
        acc = np.full(n, int(round((3 + f) * 1024)), np.int32)   # u = 3 + f (f on a 1/1024 grid)
        u = acc[0] / 1024.0
        codes = O.quantize_sr(acc, 1.0 / 1024.0, q, seed=7, iteration=1).astype(np.float64)
        assert set(np.unique(codes)) <= {np.floor(u), np.ceil(u)}
        p_up = (codes > np.floor(u)).mean()
        frac = u - np.floor(u)
        assert abs(p_up - frac) < 4.0 * np.sqrt(max(frac * (1 - frac), 1e-4) / n) + 2.0 ** -16
        assert abs(codes.mean() - u) < 0.012                     # E[q] = u


def test_saturation_and_zero_point():
    q = _state(0.0, 6.0)                                         # zero point -128
    assert q.zero_point == -128
    big = np.array([2**31 - 1, -2**31, 0], np.int32)
    assert O.quantize_sr(big, 1e20, q, 1, 1).tolist()[:2] == [127, -128]
    assert O.quantize_sr(big, 1e-3, q, 1, 1).tolist()[2] == -128  # real zero stays the zero point (u = 0 exactly)


def test_layer_uses_iteration_count_and_previous_range():
    g = np.random.default_rng(33)
    layer = O.Layer(eta=0.9, sr_seed=77)
    acc0 = g.integers(-5000, 5000, size=(16, 24)).astype(np.int32)
    r0 = layer.step(acc0, 1e-3)
    assert r0.mode == "dynamic" and layer.state.step == 1
    ref = O.Range()
    _, codes = O.dynamic_sr(acc0, 1e-3, ref, 77)
    assert np.array_equal(r0.q, codes)
    fresh = O.Range()
    O.dynamic(acc0, 1e-3, fresh)                                 # same range as the deterministic dynamic path
    assert (fresh.q_min, fresh.q_max) == (ref.q_min, ref.q_max)
    before = layer.state.copy()
    acc1 = g.integers(-9000, 9000, size=(16, 24)).astype(np.int32)
    r1 = layer.step(acc1, 1e-3)
    assert np.array_equal(r1.q, O.quantize_sr(acc1, 1e-3, before, 77, 1))   # old range, draws of iteration 1
    assert not np.array_equal(r1.q, O.quantize_sr(acc1, 1e-3, before, 77, 2))


@pytest.mark.parametrize("prior_steps", [0, 3])
def test_dynamic_path_draws_with_the_count_before_its_update(prior_steps):
    """The dynamic path with stochastic rounding is Eq. 1 for the range (the separately pinned deterministic dynamic
    path gives the same range) followed by the separately pinned static stochastic quantizer, drawing with the number
    of updates the state had seen BEFORE this call; one count later gives other codes."""
    g = np.random.default_rng(35 + prior_steps)
    acc = g.integers(-7000, 9000, size=(12, 40)).astype(np.int32)
    s_acc, seed = 2.5e-3, 4242
    st = O.derive(O.Range(q_min=-1.0, q_max=2.0, step=prior_steps))
    yf, codes = O.dynamic_sr(acc, s_acc, st, seed)
    ref = O.derive(O.Range(q_min=-1.0, q_max=2.0, step=prior_steps))
    yf_ref, _ = O.dynamic(acc, s_acc, ref)
    assert st.astuple() == ref.astuple() and st.step == prior_steps + 1
    assert (st.q_min, st.q_max) == (float(yf_ref.min()), float(yf_ref.max()))
    assert np.array_equal(yf, yf_ref)
    assert np.array_equal(codes, O.quantize_sr(acc, s_acc, st, seed, iteration=prior_steps))
    assert not np.array_equal(codes, O.quantize_sr(acc, s_acc, st, seed, iteration=prior_steps + 1))
    if prior_steps:
        assert not np.array_equal(codes, O.quantize_sr(acc, s_acc, st, seed, iteration=prior_steps - 1))
