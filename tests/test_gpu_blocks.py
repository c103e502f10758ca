"""GPU parity of the block-wise variant (Algorithm 2) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import REL, dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


class BlockLockStep:
    """Library and block-wise oracle side by side; the oracle rounds with the library's fp32 scales."""

    def __init__(self, n, offsets, x0, *, grad_dtype=pkg.GRAD_F32, payload_dtype=pkg.PAYLOAD_I32,
                 rounding=pkg.ROUND_RANDOM, beta=0.9, eps=1e-8, seed=0, fused_path=0, unaligned=False):
        self.n, self.offsets, self.d = n, list(offsets), offsets[-1]
        self.lib = pkg.IntSGD(n, self.d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding,
                              beta=beta, eps=eps, seed=seed)
        self.lib.intsgd_set_fused_path(fused_path)
        self.lib.intsgd_set_blocks(offsets)
        self.orc = oracle.OracleIntSGDBlocks(n, offsets, beta=beta, eps=eps, seed=seed, payload_dtype=payload_dtype,
                                             rounding=rounding)
        self.unaligned = unaligned
        self.x_ref = x0.copy()
        self.x_dev = self._dev(x0.copy())
        self.agg_dev = torch.zeros(self.d + 1, dtype=torch.int32, device=dev())[1 if unaligned else 0:][: self.d]

    def _dev(self, a):
        if not self.unaligned:
            return to_dev(a)
        return to_dev(np.concatenate([a[:1], a]))[1:]

    def close(self):
        self.lib.close()

    def _compare_blocks(self, got, want, what):
        for l, (g, w) in enumerate(zip(got, want)):
            assert rel_close(g, float(w)), (what, l, g, w)

    def exact(self, grads, eta):
        self.lib.intsgd_step([self._dev(g) for g in grads], self.x_dev, None, eta_k=eta, mode=pkg.MODE_EXACT)
        ref = self.orc.exact_step(grads, self.x_ref, eta)
        st = self.lib.intsgd_get_stats()
        bst = self.lib.intsgd_get_block_state()
        assert np.array_equal(to_host(self.x_dev), self.x_ref)
        self._compare_blocks(bst["dx2"], ref["dx2"], "dx2")
        assert rel_close(st["dx2"], sum(ref["dx2"])) and st["step"] == self.orc.step

    def step(self, grads, eta):
        g_dev = [self._dev(g) for g in grads]
        self.lib.intsgd_step(g_dev, self.x_dev, self.agg_dev, eta_k=eta, mode=pkg.MODE_FUSED)
        st = self.lib.intsgd_get_stats()
        bst = self.lib.intsgd_get_block_state()
        own = self.orc.scales(eta)        # the oracle's own r and alpha first (does not advance its state)
        self._compare_blocks(bst["r"], [t[0] for t in own], "r")
        self._compare_blocks(bst["alpha"], [t[2] for t in own], "alpha")
        self._compare_blocks(bst["c"], [t[3] for t in own], "c")
        ref = self.orc.int_step(grads, self.x_ref, eta,
                                alpha_c=[(np.float32(a), np.float32(c)) for a, c in zip(bst["alpha"], bst["c"])])
        assert np.array_equal(to_host(self.agg_dev), ref["agg"]), "aggregate mismatch"
        assert np.array_equal(to_host(self.x_dev).view(np.uint32), self.x_ref.view(np.uint32)), "x mismatch"
        self._compare_blocks(bst["dx2"], ref["dx2"], "dx2")
        assert rel_close(st["dx2"], sum(ref["dx2"]))
        assert st["clip_count"] == ref["clip_count"] and st["nonfinite"] == ref["nonfinite"]
        assert st["agg_overflow"] == ref["agg_overflow"] and st["max_abs_agg"] == ref["max_abs_agg"]
        assert st["step"] == self.orc.step
        return st, bst, ref


def _random_offsets(rng, d, B):
    cuts = sorted(set(int(v) for v in rng.integers(1, d, B - 1)))
    return [0] + cuts + [d]


@pytest.mark.parametrize("path,unaligned", [(0, False), (1, False), (1, True)])
@pytest.mark.parametrize("grad_dtype,payload_dtype,rounding", [
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM),
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_NEAREST), (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM16), (pkg.GRAD_BF16, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM_COMPARE)])
def test_blockwise_lockstep_with_ragged_segments(path, unaligned, grad_dtype, payload_dtype, rounding):
    """Segments of 1 to ~100k coordinates whose boundaries are not multiples of 4 or 128, a ragged
    tail, per-segment gradient scales spread over three decades."""
    rng = np.random.default_rng(5)
    d, n, eta = 3 * (1 << 17) + 7, 5, 0.1
    offsets = [0, 1, 2, 5, 64, 130, 131, 4096, 4100] + [o for o in _random_offsets(rng, d, 9)[1:-1] if o > 5000] + \
              [d - 9, d - 2, d]
    offsets = sorted(set(offsets))
    scales = 10.0 ** rng.uniform(-4, -1, len(offsets) - 1)

    def grads():
        out = []
        for _ in range(n):
            g = np.concatenate([rng.normal(0, s, b - a) for s, a, b in zip(scales, offsets, offsets[1:])]).astype(np.float32)
            out.append(synth.to_bf16_bits(g) if grad_dtype == pkg.GRAD_BF16 else g)
        return out

    ls = BlockLockStep(n, offsets, rng.normal(0, 1, d).astype(np.float32), grad_dtype=grad_dtype,
                       payload_dtype=payload_dtype, rounding=rounding, seed=21, fused_path=path, unaligned=unaligned)
    try:
        ls.exact(grads(), eta)
        for _ in range(4):
            st, bst, ref = ls.step(grads(), eta)
        # the point of the variant: every block keeps a useful integer range
        assert min(bst["alpha"]) < max(bst["alpha"]) / 50
    finally:
        ls.close()


def test_blockwise_with_values_outside_the_fast_range():
    rng = np.random.default_rng(6)
    d, n, eta = 20_001, 3, 0.1
    offsets = [0, 777, 10_003, d]
    ls = BlockLockStep(n, offsets, rng.normal(0, 1, d).astype(np.float32), payload_dtype=pkg.PAYLOAD_I8, seed=3)
    try:
        g = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        ls.exact(g, eta)
        for _ in range(3):
            g = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
            idx = rng.integers(0, d, 30)
            g[1][idx[:6]] = [np.inf, -np.inf, np.nan, 1e30, -1e30, 50.0]
            g[2][idx[6:]] *= 1e3
            g[0][d - 1] = np.nan
            st, _, _ = ls.step(g, eta)
        assert sum(st["clip_count"]) > 0 and st["nonfinite"] > 0
    finally:
        ls.close()


def test_resnet18_shaped_blocks():
    """Config 3 with its 62 per-layer segments as blocks: a few full steps, then sampled windows."""
    n, d, eta, seed = 16, synth.RESNET18_D, 0.1, 7
    offsets = [0] + list(np.cumsum(synth.RESNET18_SEGMENTS))
    offsets = [int(o) for o in offsets]
    sets = [[synth.resnet18_gradient(i, p) for i in range(n)] for p in range(2)]
    ls = BlockLockStep(n, offsets, synth.iterate(d, seed=34), seed=seed)
    try:
        ls.exact(sets[0], eta)
        for k in range(1, 3):
            st, bst, ref = ls.step(sets[k % 2], eta)
        # layers with small gradients get a large alpha of their own instead of rounding to 0 / +-1
        assert max(bst["alpha"]) / min(bst["alpha"]) > 100
        lay = np.array(synth.resnet18_layer_scales())
        assert np.argmax(bst["alpha"]) in np.argsort(lay)[:8]
    finally:
        ls.close()


def test_block_mode_api_rules():
    d = 1000
    x = torch.zeros(d, device=dev())
    g = [torch.ones(d, device=dev())]
    with pkg.IntSGD(1, d, eps=0.0) as lib:
        for bad in ([0, 10], [1, d], [0, 5, 5, d], [0, 600, 500, d]):
            with pytest.raises(pkg.IntSGDError) as e:
                lib.intsgd_set_blocks(bad)
            assert e.value.code == pkg.ERR_INVALID_ARG
        lib.intsgd_set_blocks([0, 500, d])
        for call in (lambda: lib.intsgd_sqdiff(x, x), lambda: lib.intsgd_encode(0, g[0], x),
                     lambda: lib.intsgd_aggregate(g, x), lambda: lib.intsgd_scale(0.1, 1.0),
                     lambda: lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_TWO_KERNEL, payload_scratch=g)):
            with pytest.raises(pkg.IntSGDError) as e:
                call()
            assert e.value.code == pkg.ERR_UNSUPPORTED
        # r = 0 with eps = 0 in every block: reported, nothing applied
        lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_FUSED)
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_get_stats()
        assert e.value.code == pkg.ERR_SCALE_NONFINITE
        assert float(x.abs().max()) == 0.0
        # resume: impose per-block state, step, and read it back
        lib.intsgd_set_block_state(r=[0.0, 0.0], dx2=[1e-3, 4e-3])
        lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_FUSED)
        st = lib.intsgd_get_stats()
        bst = lib.intsgd_get_block_state()
        for l, dl in enumerate((500, 500)):
            r, a64, a32, c32 = oracle.scale_block(d, dl, 1, 0.1, 0.9, 0.0, 0.0, [1e-3, 4e-3][l])
            assert bst["r"][l] == r and bst["alpha"][l] == float(a32) and bst["c"][l] == float(c32)
        assert st["step"] == 1
        lib.intsgd_set_blocks(None)                     # back to the scalar rule
        lib.intsgd_sqdiff(x, x)


def test_blockwise_norms_are_reproducible_run_to_run():
    rng = np.random.default_rng(8)
    d, n = (1 << 20) + 3, 4
    offsets = [0, 1000, 70_001, 500_000, d]
    grads = [to_dev(rng.normal(0, 1e-2, d).astype(np.float32)) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    runs = []
    for _ in range(3):
        with pkg.IntSGD(n, d, seed=4) as lib:
            lib.intsgd_set_blocks(offsets)
            x = to_dev(x0.copy())
            lib.intsgd_step(grads, x, None, eta_k=0.1, mode=pkg.MODE_EXACT)
            for _ in range(3):
                lib.intsgd_step(grads, x, None, eta_k=0.1, mode=pkg.MODE_FUSED)
            runs.append((lib.intsgd_get_block_state(), to_host(x)))
    for b, xx in runs[1:]:
        assert b["dx2"] == runs[0][0]["dx2"] and b["r"] == runs[0][0]["r"] and b["alpha"] == runs[0][0]["alpha"]
        assert np.array_equal(xx, runs[0][1])
