"""Pins for the oracle's block-wise variant (Algorithm 2 / Proposition 4 of the IntSGD paper)."""
import math

import numpy as np
import pytest

import oracle


def _grads(rng, n, d, scale=1e-2):
    return [rng.normal(0, scale, d).astype(np.float32) for _ in range(n)]


def test_one_block_is_algorithm_1():
    """B = 1: the same r, alpha equal to a few fp64 ulp (the two printed forms are algebraically
    equal), and with the same fp32 scale imposed the vectors are identical."""
    rng = np.random.default_rng(0)
    n, d, eta = 3, 1001, 0.2
    a = oracle.OracleIntSGD(n, d, seed=9)
    b = oracle.OracleIntSGDBlocks(n, [0, d], seed=9)
    xa = rng.normal(0, 1, d).astype(np.float32)
    xb = xa.copy()
    g = _grads(rng, n, d)
    a.exact_step(g, xa, eta)
    b.exact_step(g, xb, eta)
    assert np.array_equal(xa, xb) and b.dx2 == [a.dx2]
    for _ in range(4):
        g = _grads(rng, n, d)
        oa = a.int_step(g, xa, eta)
        ob = b.int_step(g, xb, eta, alpha_c=[(oa["alpha"], oa["c"])])
        assert ob["r"] == [oa["r"]]
        assert ob["alpha64"][0] == pytest.approx(oa["alpha64"], rel=1e-14)
        assert np.array_equal(oa["agg"], ob["agg"]) and np.array_equal(xa, xb)
        assert ob["dx2"] == [oa["dx2"]]


def test_per_block_scale_follows_the_printed_rule_and_its_closed_form():
    rng = np.random.default_rng(1)
    offsets = [0, 5, 6, 300, 1000, 1003]
    n, eta, beta, eps = 4, 0.1, 0.9, 1e-3
    d = offsets[-1]
    orc = oracle.OracleIntSGDBlocks(n, offsets, beta=beta, eps=eps, seed=2)
    x = rng.normal(0, 1, d).astype(np.float32)
    orc.exact_step(_grads(rng, n, d), x, eta)
    hist = [list(orc.dx2)]
    for k in range(1, 5):
        x_old = x.copy()
        out = orc.int_step(_grads(rng, n, d), x, eta)
        total = 0.0
        for l, (a, b) in enumerate(zip(offsets, offsets[1:])):
            dl = b - a
            unrolled = (1 - beta) * sum(beta**t * hist[-1 - t][l] for t in range(len(hist)))
            assert out["r"][l] == pytest.approx(unrolled, rel=1e-12)
            want = eta * math.sqrt(dl) / math.sqrt(2 * n * out["r"][l] + eta**2 * (dl / d) * eps**2)
            assert out["alpha64"][l] == pytest.approx(want, rel=1e-13)
            assert float(out["alpha"][l]) == pytest.approx(want, rel=2.0**-23)
            total += dl * eta**2 / out["alpha64"][l] ** 2
        # the error budget of Assumption 1: sum_l d_l eta^2 / alpha_l^2 = 2 n sum_l r_l + eta^2 eps^2
        assert total == pytest.approx(2 * n * sum(out["r"]) + eta**2 * eps**2, rel=1e-12)
        hist.append([oracle.sqdiff(x[a:b], x_old[a:b]) for a, b in zip(offsets, offsets[1:])])
        assert out["dx2"] == hist[-1]


def test_blocks_use_their_own_scale_and_the_absolute_random_stream():
    rng = np.random.default_rng(2)
    offsets = [0, 7, 64, 200]
    n, d, eta, seed = 2, 200, 0.5, 11
    orc = oracle.OracleIntSGDBlocks(n, offsets, seed=seed)
    x0 = rng.normal(0, 1, d).astype(np.float32)
    # block 1 has gradients 1000 x larger: a single global alpha would round block 0 to 0 / +-1
    g = _grads(rng, n, d)
    for gi in g:
        gi[7:64] *= 1000.0
    x = x0.copy()
    orc.exact_step(g, x, eta)
    x1 = x.copy()
    out = orc.int_step(g, x, eta)
    assert float(out["alpha"][1]) < float(out["alpha"][0]) / 100
    for l, (a, b) in enumerate(zip(offsets, offsets[1:])):
        xw = x1[a:b].copy()
        ref = oracle.step_window([gi[a:b] for gi in g], xw, out["alpha"][l], out["c"][l], step=1, seed=seed, j0=a)
        assert np.array_equal(ref["agg"], out["agg"][a:b]) and np.array_equal(xw, x[a:b])
        # each block keeps the magnitude bound of Section 4.2 in its own dimension
        y = np.abs(out["alpha"][l] * g[0][a:b]).max()
        assert y < 40 * math.sqrt((b - a) / (2 * n)) + 40
