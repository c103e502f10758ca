"""Pins for the oracle's IntDIANA step (Algorithm 3 of the IntSGD paper)."""
import math

import numpy as np
import pytest

import oracle
from oracle import ROUND_NEAREST


def _hand(golden_dir):
    vals = {}
    for line in (golden_dir / "diana_hand_example.txt").read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            vals[k] = np.array([float(t) for t in v], dtype=np.float32)
    return vals


def test_hand_example(golden_dir):
    h = _hand(golden_dir)
    h_local = [h["h0"].copy(), h["h1"].copy()]
    h_global, x = h["h"].copy(), h["x"].copy()
    out = oracle.diana_step_window([h["g0"], h["g1"]], h_local, h_global, x, np.float32(4.0), 0.5, step=1, seed=0,
                                   rounding=ROUND_NEAREST)
    assert list(out["agg"]) == [int(v) for v in h["q_sum"]]
    assert np.array_equal(h_local[0], h["h0_new"]) and np.array_equal(h_local[1], h["h1_new"])
    assert np.array_equal(h_global, h["h_new"]) and np.array_equal(x, h["x_new"])
    assert out["dx2"] == float(h["dx2"][0])


def test_zero_shifts_give_the_intsgd_integers_and_step():
    """h_i = h = 0: the messages are Int(alpha g_i), so the aggregate equals Algorithm 1's and the
    update agrees to fp32 rounding of eta / (n alpha)."""
    rng = np.random.default_rng(0)
    n, d, eta, alpha = 4, 3001, 0.25, np.float32(37.0)
    grads = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    xa, xb = x0.copy(), x0.copy()
    h_local = [np.zeros(d, dtype=np.float32) for _ in range(n)]
    h_global = np.zeros(d, dtype=np.float32)
    a = oracle.diana_step_window(grads, h_local, h_global, xa, alpha, eta, step=3, seed=8)
    b = oracle.step_window(grads, xb, alpha, np.float32(eta / (n * float(alpha))), step=3, seed=8)
    assert np.array_equal(a["agg"], b["agg"]) and a["clip_count"] == b["clip_count"]
    np.testing.assert_allclose(xa, xb, rtol=0, atol=2e-7 * np.abs(x0).max() + 1e-7)
    # h_i moved by the decoded message, h by their mean
    for i in range(n):
        q = oracle.encode(grads[i], alpha, worker=i, step=3, seed=8, n=n)[0]
        np.testing.assert_allclose(h_local[i], q / float(alpha), rtol=3e-7, atol=0)
    np.testing.assert_allclose(h_global, a["agg"] / (n * float(alpha)), rtol=3e-7, atol=0)


def test_global_shift_is_the_mean_of_the_local_shifts():
    rng = np.random.default_rng(1)
    n, d, eta = 5, 2000, 0.1
    orc = oracle.OracleIntDIANA(n, d, seed=3)
    x = rng.normal(0, 1, d).astype(np.float32)
    orc.exact_step([rng.normal(0, 1, d).astype(np.float32) for _ in range(n)], x, eta)
    for _ in range(10):
        orc.int_step([rng.normal(0, 1, d).astype(np.float32) for _ in range(n)], x, eta)
        mean = np.mean([h.astype(np.float64) for h in orc.h_local], axis=0)
        np.testing.assert_allclose(orc.h_global, mean, rtol=0, atol=2e-5)


def test_scale_is_proposition_3_by_default_and_a_matched_shift_sends_zeros():
    rng = np.random.default_rng(2)
    n, d, eta = 3, 512, 0.2
    orc = oracle.OracleIntDIANA(n, d, seed=1)
    x = rng.normal(0, 1, d).astype(np.float32)
    g = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]
    orc.exact_step(g, x, eta)
    norm = math.sqrt(orc.dx2)
    out = orc.int_step(g, x, eta)
    assert out["alpha64"] == pytest.approx(eta * math.sqrt(d) / (math.sqrt(2 * n) * norm), rel=1e-13)
    # g_i == h_i exactly: every message is zero, the shifts stay, x moves by eta * h
    orc.h_local = [gi.copy() for gi in g]
    h_before, x_before = orc.h_global.copy(), x.copy()
    out = orc.int_step(g, x, eta)
    assert not out["agg"].any() and out["max_abs_agg"] == 0
    assert all(np.array_equal(h, gi) for h, gi in zip(orc.h_local, g)) and np.array_equal(orc.h_global, h_before)
    assert np.array_equal(x, x_before - np.float32(eta) * h_before)


def test_heterogeneous_gradients_integers_stay_small_unlike_intsgd():
    """Section A.2 / Appendix C.5: with full gradients of heterogeneous f_i the integers of IntSGD
    grow as the iterates converge; compressing g_i - h_i keeps them bounded."""
    rng = np.random.default_rng(3)
    n, d, eta, steps = 4, 400, 0.3, 120
    b = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]     # f_i(x) = |x - b_i|^2 / 2
    grad = lambda x: [(x - bi).astype(np.float32) for bi in b]
    sgd = oracle.OracleIntSGD(n, d, beta=0.0, eps=0.0, seed=5)
    dia = oracle.OracleIntDIANA(n, d, beta=0.0, eps=0.0, seed=5)
    xs, xd = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    sgd.exact_step(grad(xs), xs, eta)
    dia.exact_step(grad(xd), xd, eta)
    big_sgd, big_dia = [], []     # largest integer a worker transmits: |alpha g_i|_inf resp. |alpha (g_i - h_i)|_inf
    for _ in range(steps):
        gs, gd = grad(xs), grad(xd)
        hd = [h.copy() for h in dia.h_local]
        a_s = float(sgd.int_step(gs, xs, eta)["alpha"])
        a_d = float(dia.int_step(gd, xd, eta)["alpha"])
        big_sgd.append(max(np.abs(a_s * g).max() for g in gs))
        big_dia.append(max(np.abs(a_d * (g - h)).max() for g, h in zip(gd, hd)))
    opt = np.mean(b, axis=0)
    assert np.abs(xd - opt).max() < 1e-3
    assert max(big_dia[20:]) <= 4 * math.sqrt(d)          # a few bits, flat
    assert big_sgd[-1] > 100 * max(big_dia[20:])          # IntSGD's messages keep growing as x converges
