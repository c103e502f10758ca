"""Pins for the optional 16-bit draw stream of the oracle (rounding mode 2)."""
import math

import numpy as np
import pytest

import oracle
from oracle import ROUND_RANDOM16

from test_oracle_philox import _philox_python

M32 = 0xFFFFFFFF


def _draw16_python(seed, step, worker, j):
    """Independent statement of the layout on Python integers."""
    u, e = divmod(j, 4)
    pair = ((u >> 10) << 9) | (u & 511)
    h = (u >> 9) & 1
    words = _philox_python([pair & M32, pair >> 32, worker, step], [seed & M32, seed >> 32])
    word = words[2 * h + e // 2]
    return ((word >> 16) if (e & 1) else (word & 0xFFFF)) / 65536.0


def test_layout_against_an_independent_statement():
    seed = 0xFEDCBA9876543210
    js = list(range(0, 40)) + [2047, 2048, 2049, 4095, 4096, 4100, 4 * 1023 + 3, 4 * 1024, 4 * 1536 + 1,
                               (1 << 34) + 5, (1 << 36) + 4 * 777 + 2]
    for (step, worker) in [(0, 0), (7, 3), (2**32 - 1, 63)]:
        for j in js:
            assert oracle.draw_uniform16(seed, step, worker, j) == _draw16_python(seed, step, worker, j)


def test_one_block_serves_eight_coordinates_and_no_bits_are_reused():
    # units u and u + 512 (u < 512 within a group of 1024) share a block; their 8 coordinates take the
    # 8 distinct half-words of it
    seed, step, worker = 5, 1, 2
    for u in (0, 3, 511, 1024 + 17, 5 * 1024 + 500):
        pair = ((u >> 10) << 9) | (u & 511)
        words = _philox_python([pair & M32, pair >> 32, worker, step], [seed & M32, seed >> 32])
        halves = sorted([w & 0xFFFF for w in words] + [w >> 16 for w in words])
        got = sorted(int(oracle.draw_uniform16(seed, step, worker, 4 * uu + e) * 65536)
                     for uu in (u, u + 512) for e in range(4))
        assert got == halves


def test_uniformity_and_independence():
    n = 1 << 15
    a = np.array([oracle.draw_uniform16(3, 1, 0, j) for j in range(n)])
    assert 0.0 <= a.min() and a.max() < 1.0 and np.all(a * 65536 == np.round(a * 65536))
    bins = np.bincount((a * 64).astype(int), minlength=64)
    chi2 = float(((bins - n / 64) ** 2 / (n / 64)).sum())
    assert 25 < chi2 < 120
    b = np.array([oracle.draw_uniform16(3, 1, 1, j) for j in range(n)])
    c = np.array([oracle.draw_uniform16(3, 2, 0, j) for j in range(n)])
    for other in (b, c, np.roll(a, 1), np.roll(a, 4), np.roll(a, 2048)):
        assert abs(np.corrcoef(a, other)[0, 1]) < 5 / math.sqrt(n)


@pytest.mark.parametrize("t", [0.25, -0.25, 3.7, -2.9, 0.5, 1.0 / 3.0])
def test_rounding_is_unbiased_to_the_draw_resolution(t):
    """P(up) = floor(p 2^16) / 2^16, so |E Int(t) - t| <= 2^-16 (zero when p is a multiple of 2^-16)."""
    N = 1 << 17
    grad = np.full(N, t, dtype=np.float32)
    q, clip, nonf = oracle.encode(grad, np.float32(1.0), worker=1, step=4, seed=99, n=4, rounding=ROUND_RANDOM16)
    t32 = float(np.float32(t))
    p = t32 - math.floor(t32)
    assert set(np.unique(q)) <= {math.floor(t32), math.floor(t32) + 1}
    assert abs(q.mean() - t32) <= 4 * math.sqrt(p * (1 - p) / N) + 2.0**-16
    # the decision is floor(t + u) with u = v 2^-16, element by element (exact in fp64: 24 + 16 bits)
    u = np.array([oracle.draw_uniform16(99, 4, 1, j) for j in range(256)])
    assert np.array_equal(q[:256], np.floor(np.float64(t32) + u).astype(int))


def test_step_with_16_bit_draws_differs_from_the_default_stream_only_in_the_draws():
    rng = np.random.default_rng(0)
    n, d = 3, 3000
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    a, b = x0.copy(), x0.copy()
    alpha, c = np.float32(9.0), np.float32(0.01)
    oa = oracle.step_window(grads, a, alpha, c, step=2, seed=7)
    ob = oracle.step_window(grads, b, alpha, c, step=2, seed=7, rounding=ROUND_RANDOM16)
    assert not np.array_equal(oa["agg"], ob["agg"])
    assert np.abs(oa["agg"] - ob["agg"]).max() <= n      # each worker differs by at most one unit
    for j0, j1 in [(0, 7), (2040, 2060), (2999, 3000)]:   # windows reproduce the full vector
        w = x0[j0:j1].copy()
        ow = oracle.step_window([g[j0:j1] for g in grads], w, alpha, c, step=2, seed=7, j0=j0, rounding=ROUND_RANDOM16)
        assert np.array_equal(ow["agg"], ob["agg"][j0:j1]) and np.array_equal(w, b[j0:j1])
