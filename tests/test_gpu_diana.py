"""GPU parity of the IntDIANA step (Algorithm 3) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


class DianaLockStep:
    def __init__(self, n, d, x0, *, grad_dtype=pkg.GRAD_F32, payload_dtype=pkg.PAYLOAD_I32,
                 rounding=pkg.ROUND_RANDOM, beta=0.0, eps=0.0, seed=0, unaligned=False, fused_path=0):
        self.n, self.d, self.unaligned = n, d, unaligned
        self.lib = pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding,
                              beta=beta, eps=eps, seed=seed)
        self.lib.intsgd_set_fused_path(fused_path)     # 0: pipelined kernel when the pointers allow it; 1: direct kernel
        self.orc = oracle.OracleIntDIANA(n, d, beta=beta, eps=eps, seed=seed, payload_dtype=payload_dtype,
                                         rounding=rounding)
        self.x_ref = x0.copy()
        self.x_dev = self._dev(x0.copy())
        self.h_dev = [self._dev(np.zeros(d, dtype=np.float32)) for _ in range(n)]
        self.hg_dev = self._dev(np.zeros(d, dtype=np.float32))
        self.agg_dev = torch.zeros(d + 1, dtype=torch.int32, device=dev())[1 if unaligned else 0:][:d]

    def _dev(self, a):
        if not self.unaligned:
            return to_dev(a)
        return to_dev(np.concatenate([a[:1], a]))[1:]

    def close(self):
        self.lib.close()

    def exact(self, grads, eta):
        self.lib.intsgd_step([self._dev(g) for g in grads], self.x_dev, None, eta_k=eta, mode=pkg.MODE_EXACT)
        self.orc.exact_step(grads, self.x_ref, eta)
        assert np.array_equal(to_host(self.x_dev), self.x_ref)

    def step(self, grads, eta):
        self.lib.intsgd_diana_step([self._dev(g) for g in grads], self.h_dev, self.hg_dev, self.x_dev, self.agg_dev,
                                   eta_k=eta)
        st = self.lib.intsgd_get_stats()
        ref = self.orc.int_step(grads, self.x_ref, eta, alpha=np.float32(st["alpha"]))
        assert rel_close(st["r"], ref["r"]) and rel_close(st["alpha"], float(ref["alpha"]))
        assert np.array_equal(to_host(self.agg_dev), ref["agg"]), "aggregate mismatch"
        for i in range(self.n):
            assert np.array_equal(to_host(self.h_dev[i]).view(np.uint32), self.orc.h_local[i].view(np.uint32)), f"h_{i}"
        assert np.array_equal(to_host(self.hg_dev).view(np.uint32), self.orc.h_global.view(np.uint32)), "h"
        assert np.array_equal(to_host(self.x_dev).view(np.uint32), self.x_ref.view(np.uint32)), "x"
        assert rel_close(st["dx2"], ref["dx2"])
        assert st["clip_count"] == ref["clip_count"] and st["nonfinite"] == ref["nonfinite"]
        assert st["agg_overflow"] == ref["agg_overflow"] and st["max_abs_agg"] == ref["max_abs_agg"]
        assert st["step"] == self.orc.step
        return st, ref


@pytest.mark.parametrize("unaligned,fused_path", [(False, 0), (False, 1), (True, 0)])
@pytest.mark.parametrize("grad_dtype,payload_dtype,rounding", [
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM),
    (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_NEAREST), (pkg.GRAD_BF16, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM16), (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM_COMPARE)])
def test_diana_lockstep_on_heterogeneous_quadratics(unaligned, fused_path, grad_dtype, payload_dtype, rounding):
    """f_i(x) = |x - b_i|^2 / 2 with different b_i (heterogeneous data), full local gradients computed
    by the harness from the library's own iterate; several tiles and a ragged tail."""
    rng = np.random.default_rng(12)
    n, d, eta = 5, 3 * (1 << 16) + 3, 0.3
    b = [rng.normal(0, 1, d).astype(np.float32) for _ in range(n)]

    def grads(x):
        out = [(x - bi).astype(np.float32) for bi in b]
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    ls = DianaLockStep(n, d, np.zeros(d, dtype=np.float32), grad_dtype=grad_dtype, payload_dtype=payload_dtype,
                       rounding=rounding, seed=31, unaligned=unaligned, fused_path=fused_path)
    try:
        ls.exact(grads(ls.x_ref), eta)
        biggest = []
        for _ in range(12):
            st, ref = ls.step(grads(ls.x_ref), eta)
            biggest.append(st["max_abs_agg"])
        # the aggregated integers stay small while x converges to the mean of the b_i
        assert max(biggest[4:]) < 4 * n * 30
    finally:
        ls.close()


@pytest.mark.parametrize("fused_path", [0, 1])
def test_diana_with_values_that_clip_and_non_finite_gradients(fused_path):
    rng = np.random.default_rng(13)
    n, d, eta = 3, 40_003, 0.1
    ls = DianaLockStep(n, d, rng.normal(0, 1, d).astype(np.float32), payload_dtype=pkg.PAYLOAD_I8, beta=0.9, eps=1e-8, seed=5,
                       fused_path=fused_path)
    try:
        ls.exact([rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)], eta)
        seen_clip = seen_nonf = 0
        for _ in range(3):
            g = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
            idx = rng.integers(0, d, 20)
            g[0][idx[:5]] = [np.inf, -np.inf, np.nan, 1e30, -1e30]
            g[1][idx[5:]] *= 1e4
            g[2][d - 1] = np.inf
            st, _ = ls.step(g, eta)
            seen_clip += sum(st["clip_count"])
            seen_nonf += st["nonfinite"]
            # keep the shifts finite for the next step (a clipped message moves h_i by at most L / alpha)
            assert all(np.isfinite(h).all() for h in ls.orc.h_local)
        assert seen_clip > 0 and seen_nonf > 0
    finally:
        ls.close()


def test_diana_api_rules():
    d = 100
    z = torch.zeros(d, device=dev())
    with pkg.IntSGD(1, d) as lib:
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_diana_step([z], [z], None, z, None, eta_k=0.1)
        assert e.value.code == pkg.ERR_INVALID_ARG
        lib.intsgd_set_blocks([0, 50, d])
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_diana_step([z], [z], z, z, None, eta_k=0.1)
        assert e.value.code == pkg.ERR_UNSUPPORTED
