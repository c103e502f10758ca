"""Pins for rounding mode 3 of the oracle: Int(t) drawn by comparing a 24-bit uniform with the fp32
fractional part (up iff u < fl32(t - floor(t)))."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import ROUND_RANDOM_COMPARE


def test_uniform24_is_the_top_24_bits():
    for w in [0, 1, 255, 256, 0xFFFFFFFF, 0x80000000, 0x12345678]:
        u = oracle.uniform24_from_word(w)
        assert u == (w >> 8) / 2.0**24 and 0.0 <= u < 1.0
    assert oracle.uniform24_from_word(0xFFFFFFFF) == 1.0 - 2.0**-24


def test_definition_against_exact_rationals():
    # dyadic t (exact in fp32, fractional part exact) x a grid of u
    for num in range(-40, 41):
        t = Fraction(num, 8)
        fl = math.floor(t)
        for k in range(0, 16):
            u = Fraction(k, 16)
            want = fl + (1 if u < t - fl else 0)
            assert oracle.int_round_compare(float(t), float(u)) == want, (t, u)


def test_half_integers_and_boundaries():
    assert oracle.int_round_compare(-1.5, 0.49) == -1
    assert oracle.int_round_compare(-1.5, 0.5) == -2       # u = p stays down
    assert oracle.int_round_compare(-0.25, 0.74) == 0
    assert oracle.int_round_compare(-0.25, 0.75) == -1
    for t in [-3.0, 0.0, 5.0, 2.0**23, -(2.0**24)]:
        for u in [0.0, 0.5, 1.0 - 2.0**-24]:
            assert oracle.int_round_compare(t, u) == int(t)


def test_fractional_part_is_taken_in_fp32():
    # y = -1e-10: floor = -1 and fl32(y + 1) = 1, so every draw goes up to 0 (the sum form keeps -1 for u = 0)
    for u in [0.0, 0.5, 1.0 - 2.0**-24]:
        assert oracle.int_round_compare(-1e-10, u) == 0
    assert oracle.int_round(-1e-10, 0.0) == -1
    # in general: the decision is u < fl32(y - floor(y)), with the subtraction rounded once
    rng = np.random.default_rng(2)
    for y in np.concatenate([rng.normal(0, 1, 2000), -np.abs(rng.normal(0, 1e-6, 500))]).astype(np.float32):
        f = np.floor(y)
        p = np.float32(y - f)
        for w in rng.integers(0, 2**32, 4):
            u = oracle.uniform24_from_word(int(w))
            assert oracle.int_round_compare(float(y), u) == int(f) + (1 if u < float(p) else 0)


@pytest.mark.parametrize("t", [0.25, -0.25, 3.7, -2.9, 0.5])
def test_unbiased_with_the_oracles_draws(t):
    N = 1 << 17
    q, clip, nonf = oracle.encode(np.full(N, t, dtype=np.float32), np.float32(1.0), worker=2, step=9, seed=1234, n=4,
                                  rounding=ROUND_RANDOM_COMPARE)
    t32 = float(np.float32(t))
    p = t32 - math.floor(t32)
    assert clip == 0 and nonf == 0
    assert set(np.unique(q)) == {math.floor(t32), math.floor(t32) + 1}
    assert abs(q.mean() - t32) <= 4 * math.sqrt(p * (1 - p) / N) + 2.0**-24
    # element by element from the stream's words
    for j in range(64):
        u = oracle.uniform24_from_word(oracle.draw_word(1234, 9, 2, j))
        assert q[j] == math.floor(t32) + (1 if u < p else 0)


def test_the_two_forms_agree_in_law_but_not_draw_by_draw():
    rng = np.random.default_rng(0)
    g = rng.normal(0, 3, 1 << 16).astype(np.float32)
    a, _, _ = oracle.encode(g, np.float32(1.0), worker=0, step=1, seed=5, n=2)
    b, _, _ = oracle.encode(g, np.float32(1.0), worker=0, step=1, seed=5, n=2, rounding=ROUND_RANDOM_COMPARE)
    assert not np.array_equal(a, b) and np.abs(a - b).max() <= 1
    for q in (a, b):
        err = q - g.astype(np.float64)
        assert abs(err.mean()) < 5 * 0.41 / math.sqrt(g.size)      # sd of the error is sqrt(1/6) for continuous inputs
        assert np.all(np.abs(err) < 1.0)
