"""Pins for the scalar lines of Algorithm 1: moving average r_k and scale alpha_k (Proposition 2)."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle


def _rows(golden_dir):
    out = []
    for line in (golden_dir / "alpha_hand_example.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            out.append([float(t) for t in line.split()])
    return out


def test_hand_example(golden_dir):
    d, n, eta = 4, 2, 0.5
    rows = _rows(golden_dir)
    assert len(rows) == 4
    for beta, eps, r_prev, dx2, r_want, inner_want, alpha_want in rows:
        r, a64, a32, c32 = oracle.scale(d, n, eta, beta, eps, r_prev, dx2)
        assert r == pytest.approx(r_want, rel=1e-15)
        assert 2 * n * r / eta**2 == pytest.approx(inner_want, rel=1e-14)
        assert a64 == pytest.approx(alpha_want, rel=1e-14)
        assert a32 == np.float32(a64)
        assert float(c32) == pytest.approx(eta / (n * float(a32)), rel=2.0**-23)


def test_fp32_alpha_of_the_first_row(golden_dir):
    _, _, a32, _ = oracle.scale(4, 2, 0.5, 0.9, 1e-8, 0.0, 0.25)
    assert a32 == np.float32(3.1622777)


def test_closed_form_invariant_and_unrolled_average():
    """Proof of Proposition 2: d eta^2 / alpha^2 = eta^2 eps^2 + 2 n r_k and
    r_k = (1 - beta) sum_t beta^t ||x^{k-t} - x^{k-t-1}||^2 (so r_0 = 0)."""
    rng = np.random.default_rng(1)
    for beta, eps in [(0.9, 1e-8), (0.0, 1e-4), (0.3, 1e-6), (0.6, 0.0)]:
        d, n = 12345, 7
        r = 0.0
        hist = []
        for k in range(1, 30):
            eta = float(rng.uniform(0.01, 2.0))
            dx2 = float(rng.uniform(1e-6, 10.0))
            hist.append(dx2)
            r, a64, a32, _ = oracle.scale(d, n, eta, beta, eps, r, dx2)
            lhs = d * eta**2 / a64**2
            rhs = eta**2 * eps**2 + 2 * n * r
            assert lhs == pytest.approx(rhs, rel=1e-13)
            unrolled = (1 - beta) * sum(beta**t * hist[-1 - t] for t in range(len(hist)))
            assert r == pytest.approx(unrolled, rel=1e-12)
            assert float(a32) == pytest.approx(a64, rel=2.0**-24)


def test_exact_rational_cross_check():
    # alpha^2 = d / (2 n r / eta^2 + eps^2) with every input dyadic: the square is an exact rational
    d, n = 1 << 20, 4
    eta, beta, eps = Fraction(1, 8), Fraction(3, 4), Fraction(1, 1 << 20)
    r_prev, dx2 = Fraction(5, 16), Fraction(9, 8)
    r_want = beta * r_prev + (1 - beta) * dx2
    alpha_sq = Fraction(d) / (2 * n * r_want / eta**2 + eps**2)
    r, a64, _, _ = oracle.scale(d, n, float(eta), float(beta), float(eps), float(r_prev), float(dx2))
    assert Fraction(r) == r_want
    assert a64 == pytest.approx(math.sqrt(alpha_sq), rel=4e-16)


def test_proposition_3_special_case():
    # beta = 0, eps = 0: alpha_k = eta sqrt(d) / (sqrt(2n) ||x^k - x^{k-1}||)
    rng = np.random.default_rng(2)
    for _ in range(50):
        d, n = int(rng.integers(1, 10**7)), int(rng.integers(1, 64))
        eta, norm = float(rng.uniform(1e-3, 5)), float(rng.uniform(1e-6, 100))
        _, a64, _, _ = oracle.scale(d, n, eta, 0.0, 0.0, 123.0, norm**2)
        assert a64 == pytest.approx(eta * math.sqrt(d) / (math.sqrt(2 * n) * norm), rel=1e-14)


def test_algorithm_2_with_one_block_equals_algorithm_1():
    rng = np.random.default_rng(4)
    for _ in range(50):
        d, n = int(rng.integers(1, 10**8)), int(rng.integers(1, 32))
        eta, beta = float(rng.uniform(1e-3, 5)), float(rng.uniform(0, 0.99))
        eps, r_prev, dx2 = 10.0 ** float(rng.uniform(-8, -4)), float(rng.uniform(0, 3)), float(rng.uniform(1e-9, 3))
        r1, a1, _, _ = oracle.scale(d, n, eta, beta, eps, r_prev, dx2)
        r2, a2, _, _ = oracle.scale_block(d, d, n, eta, beta, eps, r_prev, dx2)
        assert r1 == r2
        assert a1 == pytest.approx(a2, rel=1e-14)


def test_block_rule_closed_form():
    # Algorithm 2: sum_l d_l eta^2 / alpha_l^2 = 2 n sum_l r_l + eta^2 eps^2 (the blocks' guards add to eps^2)
    d_l = [1728, 64, 36864, 10]
    d, n, eta, beta, eps = sum(d_l), 16, 0.1, 0.9, 1e-3
    rng = np.random.default_rng(8)
    dx2 = rng.uniform(1e-8, 1e-2, len(d_l))
    total, r_sum = 0.0, 0.0
    for dl, v in zip(d_l, dx2):
        r, a64, _, _ = oracle.scale_block(d, dl, n, eta, beta, eps, 0.0, float(v))
        total += dl * eta**2 / a64**2
        r_sum += r
    assert total == pytest.approx(2 * n * r_sum + eta**2 * eps**2, rel=1e-13)


def test_safeguard_regimes():
    # r = 0: alpha = sqrt(d) / eps (the eps^2 term is the only one left)
    _, a64, a32, _ = oracle.scale(1 << 20, 4, 0.1, 0.9, 1e-8, 0.0, 0.0)
    assert a64 == pytest.approx(1024 / 1e-8, rel=1e-14)
    # r = 0 and eps = 0: the scale is infinite (callers must treat it as an error)
    _, a64, a32, _ = oracle.scale(1 << 20, 4, 0.1, 0.9, 0.0, 0.0, 0.0)
    assert math.isinf(a64) and math.isinf(float(a32))


def test_config1_expected_magnitudes():
    # d = 2^20 steps of N(0, 1e-3^2) per coordinate: ||dx||^2 ~ 1.05, r ~ 0.105, alpha ~ 112
    d, n, eta = 1 << 20, 4, 0.1
    dx2 = d * 1e-6
    r, a64, _, _ = oracle.scale(d, n, eta, 0.9, 1e-8, 0.0, dx2)
    assert r == pytest.approx(0.1048576, rel=1e-12)
    assert a64 == pytest.approx(1024 / math.sqrt(8 * 0.1048576 / 0.01), rel=1e-12)
    assert 111 < a64 < 113
