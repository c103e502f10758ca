"""Pins for the oracle's heuristic (SwitchML-style) scale, Section 5.2 of the IntSGD paper."""
import math

import numpy as np
import pytest

import oracle


def test_hand_values():
    # max 0.3 -> smallest e with 0.3 <= 2^e is -1; nb = 8, n = 4: alpha = 255 / (4 * 0.5) = 127.5
    g = [np.array([0.1, -0.3, 0.2], dtype=np.float32), np.array([0.05, 0.0, -0.25], dtype=np.float32)]
    mx, e, a, c = oracle.heuristic_scale(g + g, 4, 8, 0.5)
    assert mx == float(np.float32(0.3)) and e == -1 and a == np.float32(127.5)
    assert float(c) == pytest.approx(0.5 / (4 * 127.5), rel=2.0**-23)
    # a power of two is its own bound: max = 0.5 -> e = -1 as well; max = 0.5000001 -> e = 0
    assert oracle.heuristic_scale([np.array([0.5], dtype=np.float32)], 1, 8, 1.0)[1] == -1
    assert oracle.heuristic_scale([np.array([np.nextafter(np.float32(0.5), np.float32(1))], dtype=np.float32)], 1, 8, 1.0)[1] == 0
    assert oracle.heuristic_scale([np.array([3.0, -8.0], dtype=np.float32)], 2, 32, 1.0)[1:3] == (3, np.float32((2.0**32 - 1) / 16))


def test_no_overflow_and_at_most_one_wasted_bit():
    """The rule 'avoids overflows': n |alpha g|_inf <= 2^nb - 1, and the rounding of the exponent
    wastes less than a factor of two."""
    rng = np.random.default_rng(0)
    for _ in range(200):
        n, nb = int(rng.integers(1, 33)), int(rng.choice([8, 16, 32]))
        scale = 10.0 ** rng.uniform(-6, 3)
        grads = [rng.normal(0, scale, 257).astype(np.float32) for _ in range(n)]
        mx, e, a, c = oracle.heuristic_scale(grads, n, nb, 0.1)
        top = n * float(a) * mx
        assert top <= (2.0**nb - 1) * (1 + 1e-6)
        assert top > (2.0**nb - 1) / 2 * (1 - 1e-6)
        assert 2.0 ** (e - 1) < mx <= 2.0**e


def test_nan_is_ignored_and_degenerate_packages_have_no_scale():
    g = [np.array([np.nan, 0.25, -1.5], dtype=np.float32)]
    assert oracle.heuristic_scale(g, 1, 8, 1.0)[0] == 1.5
    assert oracle.heuristic_scale([np.zeros(4, dtype=np.float32)], 1, 8, 1.0) is None
    assert oracle.heuristic_scale([np.array([1.0, np.inf], dtype=np.float32)], 1, 8, 1.0) is None
    bits = (np.array([0.75, -2.0], dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)   # bf16 input
    assert oracle.heuristic_scale([bits], 2, 8, 1.0)[:2] == (2.0, 1)
