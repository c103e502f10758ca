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

    def step(self, grads, eta, mode=pkg.MODE_FUSED):
        g_dev = [self._dev(g) for g in grads]
        scratch = None
        if mode == pkg.MODE_TWO_KERNEL:
            pt = torch.int8 if self.orc.payload_dtype == pkg.PAYLOAD_I8 else torch.int32
            off = 1 if self.unaligned else 0
            scratch = [torch.zeros(self.d + 16, dtype=pt, device=dev())[off:off + self.d] for _ in range(self.n)]
        self.lib.intsgd_step(g_dev, self.x_dev, self.agg_dev, eta_k=eta, mode=mode, payload_scratch=scratch)
        st = self.lib.intsgd_get_stats()
        if scratch is not None:   # Algorithm 2's Int(alpha_{k,l} o g_i): every block rounded with its own scale
            bst = self.lib.intsgd_get_block_state()
            for i in range(self.n):
                got = to_host(scratch[i])
                for l, (a, b) in enumerate(zip(self.offsets, self.offsets[1:])):
                    want, _, _ = oracle.encode(grads[i][a:b], np.float32(bst["alpha"][l]), worker=i, step=self.orc.step,
                                               seed=self.orc.seed, n=self.n, payload_dtype=self.orc.payload_dtype,
                                               rounding=self.orc.rounding, j0=a)
                    assert np.array_equal(got[a:b], want), ("payload", i, l)
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


@pytest.mark.parametrize("unaligned", [False, True])
@pytest.mark.parametrize("grad_dtype,payload_dtype,rounding", [
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM),
    (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM16), (pkg.GRAD_BF16, pkg.PAYLOAD_I32, pkg.ROUND_NEAREST)])
def test_blockwise_two_kernel_step_and_payloads(unaligned, grad_dtype, payload_dtype, rounding):
    """Algorithm 2 through encode + aggregate: payloads compared per block, then aggregate, x, per-block norms and
    counters; aligned buffers take the pipelined encode, unaligned ones the direct kernels."""
    rng = np.random.default_rng(15)
    d, n, eta = (1 << 17) + 4 * 33 + 3, 4, 0.1
    offsets = sorted(set([0, 3, 130, 4097, 50_001, 2 * 4096 * 4 + 5, d - 6, d]))
    scales = 10.0 ** rng.uniform(-4, -1, len(offsets) - 1)

    def grads(plant=False):
        out = []
        for i in range(n):
            g = np.concatenate([rng.normal(0, s, b - a) for s, a, b in zip(scales, offsets, offsets[1:])]).astype(np.float32)
            if plant and i == 1:
                g[rng.integers(0, d, 5)] = [np.inf, np.nan, -1e30, 1e20, -np.inf]
                g[d - 1] = np.nan
            out.append(synth.to_bf16_bits(g) if grad_dtype == pkg.GRAD_BF16 else g)
        return out

    ls = BlockLockStep(n, offsets, rng.normal(0, 1, d).astype(np.float32), grad_dtype=grad_dtype,
                       payload_dtype=payload_dtype, rounding=rounding, seed=31, unaligned=unaligned)
    try:
        ls.exact(grads(), eta)
        for k in range(3):
            ls.step(grads(plant=(k == 1)), eta, mode=pkg.MODE_TWO_KERNEL)
        ls.step(grads(), eta, mode=pkg.MODE_FUSED)       # the two paths continue each other
    finally:
        ls.close()


def test_blockwise_separate_calls_sqdiff_scale_encode_aggregate():
    """The operator-check sequence with a partition: per-block ||x - x_prev||^2, the block scales, one encode per
    worker, one aggregate -- each call against the oracle."""
    rng = np.random.default_rng(16)
    d, n, eta, seed = 70_003, 3, 0.1, 5
    offsets = [0, 129, 4100, 33_333, d]
    x_prev = rng.normal(0, 1, d).astype(np.float32)
    x0 = (x_prev + rng.normal(0, 1e-3, d).astype(np.float32)).astype(np.float32)
    g = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
    orc = oracle.OracleIntSGDBlocks(n, offsets, seed=seed)
    for shift in (0, 1):
        with pkg.IntSGD(n, d, seed=seed) as lib:
            lib.intsgd_set_blocks(offsets)
            put = lambda a: to_dev(np.concatenate([a[:shift], a]))[shift:]
            x_dev, xp_dev = put(x0), put(x_prev)
            lib.intsgd_sqdiff(x_dev, xp_dev)
            st = lib.intsgd_get_stats()
            bst = lib.intsgd_get_block_state()
            want = [oracle.sqdiff(x0[a:b], x_prev[a:b]) for a, b in zip(offsets, offsets[1:])]
            for got, w in zip(bst["dx2"], want):
                assert rel_close(got, w, 1e-12)
            assert rel_close(st["dx2"], sum(want), 1e-12) and st["step"] == 0      # sqdiff does not advance the step
            lib.intsgd_scale(eta)
            bst = lib.intsgd_get_block_state()
            sc = orc.scales(eta, dx2=want)
            for l in range(len(offsets) - 1):
                assert rel_close(bst["r"][l], sc[l][0]) and rel_close(bst["alpha"][l], float(sc[l][2]))
            pays = [torch.zeros(d + 4, dtype=torch.int32, device=dev())[shift:shift + d] for _ in range(n)]
            for i in range(n):
                lib.intsgd_encode(i, put(g[i]), pays[i])
            agg = torch.zeros(d + 4, dtype=torch.int32, device=dev())[shift:shift + d]
            lib.intsgd_aggregate(pays, x_dev, agg)
            st = lib.intsgd_get_stats()
            bst2 = lib.intsgd_get_block_state()
            x_ref = x0.copy()
            for l, (a, b) in enumerate(zip(offsets, offsets[1:])):
                al, cl = np.float32(bst["alpha"][l]), np.float32(bst["c"][l])
                ref = oracle.step_window([gi[a:b] for gi in g], x_ref[a:b], al, cl, step=0, seed=seed, j0=a)
                assert np.array_equal(to_host(agg)[a:b], ref["agg"])
                assert rel_close(bst2["dx2"][l], ref["dx2"])
                for i in range(n):
                    want_p, _, _ = oracle.encode(g[i][a:b], al, worker=i, step=0, seed=seed, n=n, j0=a)
                    assert np.array_equal(to_host(pays[i])[a:b], want_p)
            assert np.array_equal(to_host(x_dev).view(np.uint32), x_ref.view(np.uint32))
            assert st["step"] == 1


@pytest.mark.parametrize("grad_dtype", [pkg.GRAD_F32, pkg.GRAD_BF16])
def test_blockwise_host_buffer_step_over_several_windows(grad_dtype):
    """The host-buffer step cuts the vector into windows of 2^22 coordinates; with a partition the windows share the
    block scales and their chunk partials feed one per-block norm.  Blocks straddle the window boundaries."""
    rng = np.random.default_rng(17)
    d, n, eta, seed = 2 * (1 << 22) + 4099, 2, 0.1, 8
    offsets = [0, 1000, (1 << 22) - 77, (1 << 22) + 130, 2 * (1 << 22) - 1, 2 * (1 << 22) + 4000, d]
    orc = oracle.OracleIntSGDBlocks(n, offsets, seed=seed)
    x_ref = rng.standard_normal(d, dtype=np.float32)

    def grads():
        out = [(rng.standard_normal(d, dtype=np.float32) * np.float32(1e-2)) for _ in range(n)]
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    pin = lambda a: torch.from_numpy(a.view(np.int16).copy() if a.dtype == np.uint16 else a.copy()).pin_memory()
    with pkg.IntSGD(n, d, grad_dtype=grad_dtype, seed=seed) as lib:
        lib.intsgd_set_blocks(offsets)
        hx, hagg = pin(x_ref), torch.zeros(d, dtype=torch.int32).pin_memory()
        g = grads()
        lib.intsgd_step_host([pin(a) for a in g], hx, None, eta_k=eta, mode=pkg.MODE_EXACT)
        ref = orc.exact_step(g, x_ref, eta)
        bst = lib.intsgd_get_block_state()
        assert np.array_equal(hx.numpy(), x_ref)
        for got, w in zip(bst["dx2"], ref["dx2"]):
            assert rel_close(got, w)
        for k in range(2):
            g = grads()
            lib.intsgd_step_host([pin(a) for a in g], hx, hagg, eta_k=eta, mode=pkg.MODE_FUSED)
            st = lib.intsgd_get_stats()
            bst = lib.intsgd_get_block_state()
            ref = orc.int_step(g, x_ref, eta, alpha_c=[(np.float32(a), np.float32(c)) for a, c in zip(bst["alpha"], bst["c"])])
            assert np.array_equal(hagg.numpy(), ref["agg"])
            assert np.array_equal(hx.numpy().view(np.uint32), x_ref.view(np.uint32))
            for got, w in zip(bst["dx2"], ref["dx2"]):
                assert rel_close(got, w)
            for got, w in zip(bst["r"], ref["r"]):
                assert rel_close(got, w)
            assert st["clip_count"] == ref["clip_count"] and st["max_abs_agg"] == ref["max_abs_agg"] and st["step"] == orc.step


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
        pay = [torch.zeros(d, dtype=torch.int32, device=dev())]
        # one scale per block: a single imposed dx2 or alpha has no meaning
        for call in (lambda: lib.intsgd_scale(0.1, 1.0), lambda: lib.intsgd_encode(0, g[0], pay[0], alpha_override=2.0),
                     lambda: lib.intsgd_diana_step(g, [x.clone()], x.clone(), x, None, eta_k=0.1),
                     lambda: lib.intsgd_heuristic_step(g, x, None, eta_k=0.1, num_bits=8)):
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
