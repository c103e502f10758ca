"""Pins for Int(t) (Section 2), Lemma 1 and the clipping rule of the oracle."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import PAYLOAD_I8, PAYLOAD_I32, ROUND_NEAREST


def test_int_of_integers_is_identity():
    for t in [-1000.0, -3.0, -1.0, 0.0, 1.0, 2.0, 77.0, 2.0**23, -(2.0**24)]:
        for u in [0.0, 0.3, 1.0 - 2.0**-24]:
            assert oracle.int_round(t, u) == int(t)


def test_int_definition_against_exact_rationals():
    # brute force: dyadic t (exact in fp32) x a grid of u; Int(t) = floor(t + u) in Fractions
    for num in range(-40, 41):
        t = Fraction(num, 8)
        for k in range(0, 16):
            u = Fraction(k, 16)
            want = math.floor(t + u)
            assert oracle.int_round(float(t), float(u)) == want, (t, u)
            # the same event stated on the fractional part: up iff u >= 1 - (t - floor(t))
            assert want == math.floor(t) + (1 if u >= 1 - (t - math.floor(t)) else 0)


def test_floor_of_the_unrounded_sum_on_adversarial_values():
    """t + u is never rounded before the floor: random and near-integer fp32 values with draws on
    the 2^-32 grid, against exact rational arithmetic."""
    rng = np.random.default_rng(8)
    ts = [np.float32(v) for v in rng.normal(0, 100, 3000)] + [np.float32(v) for v in rng.normal(0, 1e-3, 500)]
    for base in [1.0, -1.0, 100.0, -100.0, 4096.0, 2.0**20, -(2.0**22), 0.0]:
        b = np.float32(base)
        for _ in range(6):
            ts += [b]
            b = np.nextafter(b, np.float32(-np.inf), dtype=np.float32)
        b = np.float32(base)
        for _ in range(6):
            b = np.nextafter(b, np.float32(np.inf), dtype=np.float32)
            ts += [b]
    ts += [np.float32(v) for v in [1e-10, -1e-10, 1e-38, -1e-38, 1e-45, -1e-45, 2.0**-28, -(2.0**-28), 2.0**-29, 2.0**-24, -(2.0**-24)]]
    words = [0, 1, 2, 255, 256, 2**15 - 1, 2**24 - 1, 2**24, 2**31, 2**32 - 256, 2**32 - 1] + \
            [int(w) for w in rng.integers(0, 2**32, 24)]
    us = [oracle.uniform_from_word(w) for w in words]
    for t in ts:
        ft = Fraction(float(t))
        for u in us:
            assert oracle.int_round(float(t), u) == math.floor(ft + Fraction(u)), (float(t), u)
        # the complement of the fractional part, and its fp32 neighbours, as draws (when they are valid draws)
        need = 1 - (ft - math.floor(ft))
        for cand in [np.float32(float(need))]:
            for u in [np.nextafter(cand, np.float32(0)), cand, np.nextafter(cand, np.float32(2))]:
                if 0 <= float(u) < 1:
                    assert oracle.int_round(float(t), float(u)) == math.floor(ft + Fraction(float(u))), (float(t), float(u))


def test_negative_half_integers():
    # Int(-1.5) is -2 or -1, each with probability 1/2: floor is toward minus infinity
    assert oracle.int_round(-1.5, 0.49) == -2
    assert oracle.int_round(-1.5, 0.5) == -1
    assert oracle.int_round(-0.25, 0.24) == -1
    assert oracle.int_round(-0.25, 0.25) == 0
    assert oracle.int_round(0.75, 0.24) == 0
    assert oracle.int_round(0.75, 0.25) == 1


def test_error_strictly_below_one_everywhere():
    rng = np.random.default_rng(3)
    t = np.concatenate([rng.normal(0, 50, 4000), rng.normal(0, 1e-3, 1000), rng.normal(0, 1e5, 1000)]).astype(np.float32)
    u = rng.random(t.size).astype(np.float32)
    for ti, ui in zip(t, u):
        q = oracle.int_round(float(ti), float(ui))
        assert abs(q - float(ti)) < 1.0
        assert q in (math.floor(float(ti)), math.floor(float(ti)) + 1)


@pytest.mark.parametrize("t", [0.25, -0.25, 3.7, -2.9, 0.001, 126.5, -1e-3, 0.5])
def test_unbiased_and_variance_monte_carlo(t):
    """Lemma 1: E Int(t) = t and Var Int(t) = p(1-p) <= 1/4, with the oracle's own Philox draws."""
    N = 1 << 17
    alpha = np.float32(1.0)
    grad = np.full(N, t, dtype=np.float32)
    q, clip, nonf = oracle.encode(grad, alpha, worker=2, step=9, seed=1234, n=4)
    assert clip == 0 and nonf == 0
    t32 = float(np.float32(t))
    p = t32 - math.floor(t32)
    sd = math.sqrt(p * (1 - p) / N)
    assert abs(q.mean() - t32) <= 4 * sd + 2.0**-24
    if p not in (0.0,):
        assert q.min() != q.max()      # both outcomes occur
    assert set(np.unique(q)) <= {math.floor(t32), math.floor(t32) + 1}
    assert q.var() <= 0.25 + 1e-12
    assert abs(q.var() - p * (1 - p)) < 0.01


def test_lemma1_vector_variance_bound():
    """E || Q(x) - x ||^2 <= d / (4 alpha^2) for a scalar alpha (Lemma 1, second line)."""
    d, alpha = 1 << 15, np.float32(3.0)
    rng = np.random.default_rng(0)
    x = rng.normal(0, 1, d).astype(np.float32)
    errs = []
    for step in range(8):
        q, _, _ = oracle.encode(x, alpha, worker=0, step=step, seed=77, n=2)
        Q = q.astype(np.float64) / float(alpha)
        errs.append(float(((Q - (np.float32(alpha) * x).astype(np.float64) / float(alpha)) ** 2).sum()))
    bound = d / (4 * float(alpha) ** 2)
    mean = np.mean(errs)
    # for continuous inputs E p(1-p) = 1/6, so the mean sits near (2/3) * bound and below it
    assert mean <= bound
    assert 0.5 * bound < mean


def test_huge_values_round_to_themselves():
    # no fractional bits at or above 2^23: p = 0 and Int(y) = y for every draw
    for y in [2.0**23, 2.0**23 + 1, 2.0**27 - 8, -(2.0**26) - 8]:
        for u in [0.0, 0.999]:
            assert oracle.int_round(y, u) == int(y)


def test_tiny_values_are_not_rounded_away():
    # y = -1e-10: floor = -1; any positive draw lifts the sum above 0, the zero draw does not
    assert oracle.int_round(-1e-10, 0.0) == -1
    for u in [2.0**-32, 0.5, 1.0 - 2.0**-24]:
        assert oracle.int_round(-1e-10, u) == 0
    # y = +1e-10 never reaches 1: the largest draw is 1 - 2^-24
    for u in [0.0, 0.5, 1.0 - 2.0**-24]:
        assert oracle.int_round(1e-10, u) == 0


def test_nearest_even():
    cases = {0.5: 0, 1.5: 2, 2.5: 2, -0.5: 0, -1.5: -2, 0.49: 0, 0.51: 1, -2.51: -3, 3.0: 3}
    for y, want in cases.items():
        assert oracle.int_round_nearest(y) == want
    g = np.array(list(cases.keys()), dtype=np.float32)
    q, clip, _ = oracle.encode(g, np.float32(1.0), worker=0, step=0, seed=0, n=1, rounding=ROUND_NEAREST)
    assert list(q) == list(cases.values()) and clip == 0


def test_limit_as_float():
    assert oracle.limit_as_float(127) == 127.0
    assert oracle.limit_as_float(2**31 - 1) == 2.0**31 - 128          # largest fp32 below 2^31
    assert oracle.limit_as_float((2**31 - 1) // 16) == 2.0**27 - 8    # 2^27 - 1 is not an fp32
    assert oracle.limit_as_float(2**24) == 2.0**24
    assert oracle.limit_as_float(2**24 + 1) == 2.0**24


def test_clip_counts_closed_form_int8():
    L = 127
    alpha = np.float32(2.0)
    g = np.zeros(64, dtype=np.float32)
    g[3] = 63.5      # y = 127 exactly: not clipped
    g[4] = 63.75     # y = 127.5: clipped to 127
    g[5] = -64.0     # y = -128: clipped to -127
    g[6] = np.inf
    g[7] = -np.inf
    g[8] = np.nan
    g[9] = 3.0e38    # alpha * g overflows to +inf
    q, clip, nonf = oracle.encode(g, alpha, worker=0, step=0, seed=0, n=8, payload_dtype=PAYLOAD_I8)
    assert q.dtype == np.int8
    assert clip == 6 and nonf == 4
    assert list(q[3:10]) == [127, 127, -127, 127, -127, 0, 127]
    assert not q[:3].any() and not q[10:].any()


def test_clip_is_independent_of_the_draw_and_keeps_values_in_range():
    rng = np.random.default_rng(5)
    g = rng.normal(0, 100, 4096).astype(np.float32)
    alpha = np.float32(1.0)
    y = alpha * g
    want = int((np.abs(y) > 127).sum())
    for step in range(3):
        q, clip, _ = oracle.encode(g, alpha, worker=1, step=step, seed=3, n=2, payload_dtype=PAYLOAD_I8)
        assert clip == want
        assert q.min() >= -127 and q.max() <= 127
        inside = np.abs(y) <= 127
        assert np.all(np.abs(q[inside].astype(np.float64) - y[inside]) < 1.0)
        assert np.all(q[y > 127] == 127) and np.all(q[y < -127] == -127)


def test_default_int32_limit_makes_the_sum_fit():
    for n in [1, 2, 3, 16, 100]:
        L = oracle.default_clip_limit(n, PAYLOAD_I32)
        assert n * L <= 2**31 - 1 < n * (L + 1)
        g = np.array([3.0e9, -3.0e9, 1.0], dtype=np.float32)
        q, clip, _ = oracle.encode(g, np.float32(1.0), worker=0, step=0, seed=0, n=n)
        Lf = oracle.limit_as_float(L)
        assert clip == 2 and q[0] == int(Lf) and q[1] == -int(Lf) and q[2] == 1
        assert n * int(Lf) <= 2**31 - 1


def test_non_finite_values_on_the_int32_wire():
    # NaN -> 0, +-Inf -> +-Lf, each counted as clipped and as non-finite
    n = 4
    Lf = int(oracle.limit_as_float(oracle.default_clip_limit(n, PAYLOAD_I32)))
    g = np.array([np.nan, np.inf, -np.inf, 1.0, -np.nan], dtype=np.float32)
    q, clip, nonf = oracle.encode(g, np.float32(1.0), worker=0, step=0, seed=0, n=n)
    assert list(q) == [0, Lf, -Lf, 1, 0] and clip == 4 and nonf == 4
