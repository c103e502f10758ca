"""Pins for the vector part of Algorithm 1 in the oracle: encode, aggregate, decode, update."""
import math
from fractions import Fraction
from itertools import product

import numpy as np
import pytest

import oracle
from oracle import PAYLOAD_I8, PAYLOAD_I32, ROUND_NEAREST


def _hand(golden_dir):
    vals = {}
    for line in (golden_dir / "step_hand_example.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            vals[k] = [float(t) for t in v]
    return vals


def test_hand_example(golden_dir):
    h = _hand(golden_dir)
    alpha, n, eta = np.float32(1.0), 2, 0.5
    payloads = []
    for i in range(n):
        q, clip, nonf = oracle.encode(np.array(h[f"g{i}"], dtype=np.float32), alpha, worker=i, step=1,
                                      seed=0, n=n, u_inject=np.array(h[f"u{i}"], dtype=np.float32))
        assert list(q) == [int(v) for v in h[f"q{i}"]]
        assert clip == 0 and nonf == 0
        payloads.append(q)
    x = np.zeros(4, dtype=np.float32)
    c = np.float32(eta / (n * float(alpha)))
    agg, dx2, ovf, mx = oracle.aggregate(payloads, x, c)
    assert list(agg) == [int(v) for v in h["S"]]
    assert list(x) == h["x_new"]
    assert dx2 == h["dx2"][0]
    assert ovf == 0 and mx == 1
    _, a64, _, _ = oracle.scale(4, n, eta, 0.0, 0.0, 0.0, dx2)
    assert a64 == pytest.approx(h["next_alpha"][0], rel=1e-15)


def test_brute_force_tiny_against_exact_rationals():
    """d <= 3, n <= 2, dyadic inputs (every fp32 operation exact): enumerate a grid of draws and
    redo the whole step in exact rational arithmetic."""
    alpha = Fraction(4)
    eta = Fraction(1, 2)
    grid_g = [Fraction(k, 16) for k in (-37, -8, -3, 0, 5, 16, 29)]
    grid_u = [Fraction(k, 8) for k in range(8)]
    count = 0
    for n in (1, 2):
        c = eta / (n * alpha)
        for g in product(grid_g, repeat=n):
            for u in product(grid_u, repeat=n):
                S = 0
                for gi, ui in zip(g, u):
                    S += math.floor(alpha * gi + ui)      # Int(t) = floor(t + u)
                x0 = Fraction(3, 4)
                x_want = x0 - c * S
                payloads = []
                for i in range(n):
                    q, _, _ = oracle.encode(np.array([g[i]] * 3, dtype=np.float32), np.float32(alpha),
                                            worker=i, step=0, seed=0, n=n,
                                            u_inject=np.array([u[i]] * 3, dtype=np.float32))
                    payloads.append(q)
                x = np.full(3, float(x0), dtype=np.float32)
                agg, dx2, _, mx = oracle.aggregate(payloads, x, np.float32(c))
                assert list(agg) == [S] * 3
                assert all(Fraction(float(v)) == x_want for v in x)
                assert Fraction(dx2) == 3 * (c * S) ** 2
                assert mx == abs(S)
                count += 1
    assert count > 3000


def test_decode_identity():
    """(1/(n alpha)) sum_i Int(alpha g_i) = (1/n) sum_i Q(g_i) (display below Eq. 2)."""
    rng = np.random.default_rng(0)
    n, d, alpha = 5, 2048, np.float32(37.5)
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    qs = [oracle.encode(g, alpha, worker=i, step=4, seed=9, n=n)[0] for i, g in enumerate(grads)]
    lhs = np.sum([q.astype(np.float64) for q in qs], axis=0) / (n * float(alpha))
    rhs = np.mean([q.astype(np.float64) / float(alpha) for q in qs], axis=0)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-14, atol=1e-15)
    x = np.zeros(d, dtype=np.float32)
    eta = 1.0
    agg, _, _, _ = oracle.aggregate(qs, x, np.float32(eta / (n * float(alpha))))
    assert np.array_equal(agg, np.sum([q.astype(np.int64) for q in qs], axis=0))
    np.testing.assert_allclose(-x.astype(np.float64), lhs, rtol=3e-7, atol=1e-15)


def test_step_within_the_papers_error_bound_of_exact_sgd():
    """|x_new - (x - eta * mean g)|_inf < eta / alpha (+ fp32 slack): each Int is within 1 of its
    argument, summed over n workers and divided by n alpha."""
    rng = np.random.default_rng(1)
    n, d, eta = 8, 1 << 14, 0.3
    grads = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    for alpha in [np.float32(10.0), np.float32(1000.0), np.float32(1e5)]:
        x = x0.copy()
        c = np.float32(eta / (n * float(alpha)))
        out = oracle.step_window(grads, x, alpha, c, step=3, seed=5)
        exact = x0.astype(np.float64) - eta * np.mean([g.astype(np.float64) for g in grads], axis=0)
        err = np.abs(x.astype(np.float64) - exact).max()
        assert err < eta / float(alpha) + 4e-7
        # mean-square error of the estimator: E ||g~ - gbar||^2 <= d / (4 n alpha^2)
        gt = out["agg"].astype(np.float64) / (n * float(alpha))
        gbar = np.mean([(alpha * g).astype(np.float64) / float(alpha) for g in grads], axis=0)
        mse = float(((gt - gbar) ** 2).sum())
        bound = d / (4 * n * float(alpha) ** 2)
        assert mse < 1.15 * bound
        if float(alpha) >= 1000:   # fractional parts spread evenly: E p(1-p) = 1/6 = (2/3)(1/4)
            assert mse > 0.55 * bound
    # as alpha grows the step tends to the plain mean-gradient axpy
    assert err < 1e-5


def test_exact_first_step_is_mean_gradient_axpy():
    rng = np.random.default_rng(2)
    n, d, eta = 6, 4099, 0.25
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    x = x0.copy()
    dx2 = oracle.exact_step(grads, x, eta)
    want = x0.astype(np.float64) - eta * np.mean([g.astype(np.float64) for g in grads], axis=0)
    np.testing.assert_allclose(x, want, rtol=0, atol=2e-6)
    # the difference that feeds r_k is the fp32 difference of the stored iterates, squared in fp64
    assert dx2 == pytest.approx(float(((x - x0).astype(np.float64) ** 2).sum()), rel=1e-12)
    # one worker, eta = 1, power-of-two data: exact
    x = np.array([1.0, 2.0], dtype=np.float32)
    assert oracle.exact_step([np.array([0.5, -4.0], dtype=np.float32)], x, 1.0) == 0.25 + 16.0
    assert list(x) == [0.5, 6.0]


def test_sqdiff_and_dx2_agree_with_numpy_fp64():
    rng = np.random.default_rng(3)
    a = rng.normal(0, 1, 10007).astype(np.float32)
    b = (a + rng.normal(0, 1e-3, a.size)).astype(np.float32)
    want = float((((a - b).astype(np.float64)) ** 2).sum())
    assert oracle.sqdiff(a, b) == pytest.approx(want, rel=1e-13)
    assert oracle.sqdiff(a, a) == 0.0


def test_windows_reproduce_the_full_vector():
    """The stream is indexed by absolute coordinate, so any window can be recomputed alone."""
    rng = np.random.default_rng(4)
    n, d = 3, 1003
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    alpha, c = np.float32(20.0), np.float32(0.1 / (3 * 20.0))
    xf = x0.copy()
    full = oracle.step_window(grads, xf, alpha, c, step=7, seed=42)
    for j0, j1 in [(0, 5), (5, 6), (6, 517), (517, 1003), (1001, 1003)]:
        xw = x0[j0:j1].copy()
        w = oracle.step_window([g[j0:j1] for g in grads], xw, alpha, c, step=7, seed=42, j0=j0)
        assert np.array_equal(w["agg"], full["agg"][j0:j1])
        assert np.array_equal(xw, xf[j0:j1])
    # and step_window is the composition of encode and aggregate
    pay = [oracle.encode(g, alpha, worker=i, step=7, seed=42, n=n)[0] for i, g in enumerate(grads)]
    x2 = x0.copy()
    agg, dx2, _, mx = oracle.aggregate(pay, x2, c)
    assert np.array_equal(agg, full["agg"]) and np.array_equal(x2, xf)
    assert dx2 == full["dx2"] and mx == full["max_abs_agg"]


def test_bf16_gradients_are_widened_exactly():
    rng = np.random.default_rng(5)
    g32 = rng.normal(0, 1, 513).astype(np.float32)
    bits = (g32.view(np.uint32) >> 16).astype(np.uint16)          # truncate to bf16 bit patterns
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    a, _, _ = oracle.encode(bits, np.float32(9.0), worker=1, step=2, seed=3, n=4)
    b, _, _ = oracle.encode(widened, np.float32(9.0), worker=1, step=2, seed=3, n=4)
    assert np.array_equal(a, b)


def test_int8_aggregate_overflow_count_and_max():
    n = 3
    pay = [np.array([127, 100, -127, 40, 0], dtype=np.int8),
           np.array([127, 27, -127, 40, 0], dtype=np.int8),
           np.array([127, 0, -1, 48, 0], dtype=np.int8)]
    x = np.zeros(5, dtype=np.float32)
    agg, dx2, ovf, mx = oracle.aggregate(pay, x, np.float32(1.0))
    assert list(agg) == [381, 127, -255, 128, 0]
    assert ovf == 3 and mx == 381
    assert list(x) == [-381.0, -127.0, 255.0, -128.0, 0.0]


def test_deterministic_rounding_step():
    rng = np.random.default_rng(6)
    n, d = 4, 777
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    x = np.zeros(d, dtype=np.float32)
    alpha = np.float32(8.0)
    out = oracle.step_window(grads, x, alpha, np.float32(1.0), step=0, seed=0, rounding=ROUND_NEAREST)
    want = np.sum([np.rint((alpha * g).astype(np.float32)).astype(np.int64) for g in grads], axis=0)
    assert np.array_equal(out["agg"], want)


def test_state_machine_follows_algorithm_1_order():
    """Step 0 exact; step k >= 1 uses r_k built from the previous step length (r_0 = 0)."""
    rng = np.random.default_rng(7)
    n, d, eta = 4, 256, 0.1
    orc = oracle.OracleIntSGD(n, d, beta=0.9, eps=1e-8, seed=1)
    x = rng.normal(0, 1, d).astype(np.float32)
    hist = []
    grads = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
    x_prev = x.copy()
    orc.exact_step(grads, x, eta)
    hist.append(oracle.sqdiff(x, x_prev))
    assert orc.dx2 == hist[-1] and orc.r == 0.0 and orc.step == 1
    for k in range(1, 6):
        grads = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        x_prev = x.copy()
        out = orc.int_step(grads, x, eta)
        unrolled = 0.1 * sum(0.9**t * hist[-1 - t] for t in range(len(hist)))
        assert out["r"] == pytest.approx(unrolled, rel=1e-12)
        assert float(out["alpha"]) == pytest.approx(math.sqrt(d) / math.sqrt(2 * n * out["r"] / eta**2 + 1e-16), rel=1e-7)
        hist.append(oracle.sqdiff(x, x_prev))
        assert out["dx2"] == hist[-1]
        assert orc.step == k + 1
        # regime of Section 4.2: |alpha g|_inf <= sqrt(d / 2n) up to the moving-average factor
        assert out["max_abs_agg"] <= n * (math.sqrt(d / (2 * n)) / math.sqrt(0.1) + 1) * 4
