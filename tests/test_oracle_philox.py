"""Pins for the oracle's random stream: Philox4x32-10 and the (seed, step, worker, index) layout."""
from fractions import Fraction

import numpy as np

import oracle

M32 = 0xFFFFFFFF


def _philox_python(ctr, key, rounds=10):
    """Second, independent statement of Philox4x32 (Salmon et al., SC'11) on Python integers:
    written round-function-first with tuple rebuilds rather than the oracle's scalar updates."""
    def round_fn(c, k):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        return ((p1 >> 32) ^ c[1] ^ k[0], p1 & M32, (p0 >> 32) ^ c[3] ^ k[1], p0 & M32)

    c, k = tuple(ctr), tuple(key)
    for _ in range(rounds):
        c = round_fn(c, k)
        k = ((k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32)
    return c


def _read_kat(golden_dir):
    rows = []
    for line in (golden_dir / "philox4x32_10_kat.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], tuple(w[6:10])))
    return rows


def test_known_answer_vectors(golden_dir):
    rows = _read_kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert oracle.philox4x32_10(ctr, key) == want
        assert _philox_python(ctr, key) == want


def test_two_implementations_agree_on_random_counters():
    rng = np.random.default_rng(7)
    for _ in range(2000):
        ctr = [int(v) for v in rng.integers(0, 2**32, size=4)]
        key = [int(v) for v in rng.integers(0, 2**32, size=2)]
        assert oracle.philox4x32_10(ctr, key) == _philox_python(ctr, key)


def test_round_count_matters():
    # nine or eleven rounds give other words: the "10" is pinned by the known answers
    ctr, key = [1, 2, 3, 4], [5, 6]
    ten = _philox_python(ctr, key, 10)
    assert oracle.philox4x32_10(ctr, key) == ten
    assert _philox_python(ctr, key, 9) != ten and _philox_python(ctr, key, 11) != ten


def test_stream_layout():
    """key = (seed lo, seed hi); counter = (b lo, b hi, worker, step), b = j // 4; word j % 4."""
    seed = 0x0123456789ABCDEF
    for (step, worker, j) in [(0, 0, 0), (3, 5, 7), (2**32 - 1, 63, 2**34 + 9), (17, 1, 4 * 2**32 + 2)]:
        b = j // 4
        words = _philox_python([b & M32, b >> 32, worker, step], [seed & M32, seed >> 32])
        assert oracle.draw_word(seed, step, worker, j) == words[j % 4]


def test_uniform_from_word_is_the_word_truncated_to_fp32():
    """u = w * 2^-32 rounded toward zero to fp32: u <= w / 2^32 < next fp32 above u, and u < 1."""
    rng = np.random.default_rng(4)
    words = [0, 1, 255, 256, 0xFFFFFF, 0x1000000, 0x1000001, 0x1FFFFFF, 0xFFFFFFFF, 0xFFFFFF00, 0xFFFFFF7F,
             0x80000000, 0x800000FF, 0x12345678] + [int(w) for w in rng.integers(0, 2**32, 2000)]
    for w in words:
        u = oracle.uniform_from_word(w)
        assert np.float32(u) == u and 0.0 <= u < 1.0
        exact = Fraction(w, 2**32)
        above = float(np.nextafter(np.float32(u), np.float32(2.0)))
        assert Fraction(u) <= exact < Fraction(above), hex(w)
    assert oracle.uniform_from_word(0xFFFFFFFF) == 1.0 - 2.0**-24
    assert oracle.uniform_from_word(0xFFFFFF) == 0xFFFFFF / 2.0**32      # 24 significant bits: kept whole
    assert oracle.uniform_from_word(0x1FFFFFF) == 0x1FFFFFE / 2.0**32    # 25 bits: the lowest one dropped


def _draws(seed, step, worker, count, j0=0):
    return np.array([oracle.draw_word(seed, step, worker, j0 + j) for j in range(count)], dtype=np.uint64)


def test_uniformity_chi_square():
    # 2^16 draws into 64 bins by the word's top 6 bits: chi-square with 63 dof, mean 63, sd ~11.2
    w = _draws(seed=11, step=1, worker=0, count=1 << 16)
    bins = np.bincount((w >> 26).astype(np.int64), minlength=64)
    expect = (1 << 16) / 64
    chi2 = float(((bins - expect) ** 2 / expect).sum())
    assert 25.0 < chi2 < 120.0
    # every bit of the word is balanced (|mean - 1/2| < 5 sigma)
    for bit in range(0, 32):
        frac = float(((w >> bit) & 1).mean())
        assert abs(frac - 0.5) < 5 * 0.5 / np.sqrt(len(w))


def test_streams_differ_across_worker_step_seed_and_are_uncorrelated():
    n = 1 << 14
    base = _draws(5, 2, 3, n).astype(np.float64) / 2**32
    for other in (_draws(5, 2, 4, n), _draws(5, 3, 3, n), _draws(6, 2, 3, n), _draws(5, 2, 3, n, j0=n)):
        o = other.astype(np.float64) / 2**32
        assert not np.array_equal(o, base)
        corr = np.corrcoef(base, o)[0, 1]
        assert abs(corr) < 5 / np.sqrt(n)
    # the same key reproduces the same words (counter-based: no hidden state)
    assert np.array_equal(_draws(5, 2, 3, 64), _draws(5, 2, 3, 64))
