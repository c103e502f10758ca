"""Shared helpers of the GPU parity tests: lock-step comparison of the CUDA library with the oracle.

Lock-step protocol: the library's norm reduction is a tree, the oracle's a serial sum, so r_k and
alpha_k agree to rounding of the fp64 sum only.  Each step the oracle computes its own r_k and
alpha_k, they are compared at 1e-6 relative, and the oracle then rounds with the library's fp32
(alpha_k, c_k) so that every vector output can be compared bit for bit.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2102_08374_b200 as pkg

REL = 1e-6   # tolerance on r_k, alpha_k and dx2 (stated by the benchmark definition)


def dev():
    return torch.device("cuda:0")


def to_dev(a: np.ndarray):
    if a.dtype == np.uint16:   # bf16 bit patterns
        return torch.from_numpy(a.view(np.int16)).to(dev()).view(torch.bfloat16)
    return torch.from_numpy(a).to(dev())


def to_host(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def rel_close(a, b, rel=REL):
    return abs(a - b) <= rel * max(abs(a), abs(b), 1e-300)


class LockStep:
    """Runs the library and the oracle side by side on full vectors."""

    def __init__(self, n, d, *, grad_dtype=pkg.GRAD_F32, payload_dtype=pkg.PAYLOAD_I32,
                 rounding=pkg.ROUND_RANDOM, beta=0.9, eps=1e-8, seed=0, clip_limit=0, x0=None, fused_path=0):
        self.n, self.d = n, d
        self.lib = pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding,
                              beta=beta, eps=eps, seed=seed, clip_limit=clip_limit)
        self.lib.intsgd_set_fused_path(fused_path)
        self.orc = oracle.OracleIntSGD(n, d, beta=beta, eps=eps, seed=seed, payload_dtype=payload_dtype,
                                       clip_limit=clip_limit or None, rounding=rounding)
        self.x_ref = np.ascontiguousarray(x0, dtype=np.float32).copy()
        self.x_dev = to_dev(self.x_ref.copy())
        self.agg_dev = torch.empty(d, dtype=torch.int32, device=dev())
        pay_t = torch.int8 if payload_dtype == pkg.PAYLOAD_I8 else torch.int32
        self._pay_t = pay_t
        self.scratch = None

    def close(self):
        self.lib.close()

    def _scratch(self):
        if self.scratch is None:
            self.scratch = [torch.empty(self.d, dtype=self._pay_t, device=dev()) for _ in range(self.n)]
        return self.scratch

    def exact(self, grads, eta):
        g_dev = [to_dev(g) for g in grads]
        self.lib.intsgd_step(g_dev, self.x_dev, None, eta_k=eta, mode=pkg.MODE_EXACT)
        ref = self.orc.exact_step(grads, self.x_ref, eta)
        st = self.lib.intsgd_get_stats()
        assert np.array_equal(to_host(self.x_dev), self.x_ref)
        assert rel_close(st["dx2"], ref["dx2"])
        assert st["step"] == self.orc.step
        return st

    def step(self, grads, eta, mode=pkg.MODE_FUSED, g_dev=None, want_agg=True):
        g_dev = g_dev if g_dev is not None else [to_dev(g) for g in grads]
        agg = self.agg_dev if want_agg else None
        if mode == pkg.MODE_TWO_KERNEL:
            self.lib.intsgd_step(g_dev, self.x_dev, agg, eta_k=eta, mode=mode, payload_scratch=self._scratch())
        else:
            self.lib.intsgd_step(g_dev, self.x_dev, agg, eta_k=eta, mode=mode)
        st = self.lib.intsgd_get_stats()
        # oracle: own scalars first, compared at 1e-6; then the library's fp32 scale for the vectors
        ref = self.orc.int_step(grads, self.x_ref, eta, alpha_c=(np.float32(st["alpha"]), np.float32(st["c"])))
        assert rel_close(st["r"], ref["r"]), (st["r"], ref["r"])
        assert rel_close(st["alpha"], float(ref["alpha"])), (st["alpha"], ref["alpha"])
        assert rel_close(st["c"], float(ref["c"]))
        if want_agg:
            assert np.array_equal(to_host(self.agg_dev), ref["agg"]), "aggregate mismatch"
        x_gpu = to_host(self.x_dev)
        assert np.array_equal(x_gpu.view(np.uint32), self.x_ref.view(np.uint32)), "x mismatch (0 ULP required)"
        assert rel_close(st["dx2"], ref["dx2"]), (st["dx2"], ref["dx2"])
        assert st["clip_count"] == ref["clip_count"], (st["clip_count"], ref["clip_count"])
        assert st["nonfinite"] == ref["nonfinite"]
        assert st["agg_overflow"] == ref["agg_overflow"]
        assert st["max_abs_agg"] == ref["max_abs_agg"]
        assert st["step"] == self.orc.step
        if mode == pkg.MODE_TWO_KERNEL:
            self.last_payloads = [to_host(p) for p in self.scratch]
        return st, ref


def check_window(lib_stats, grads_dev, x_before_dev, x_after_dev, agg_dev, j0, j1, *, step, seed, n,
                 payload_dtype=pkg.PAYLOAD_I32, rounding=pkg.ROUND_RANDOM, clip_limit=None):
    """Recompute coordinates [j0, j1) of one step with the oracle and compare bit for bit."""
    grads = [to_host(g[j0:j1]) for g in grads_dev]
    xw = to_host(x_before_dev[j0:j1]).copy()
    ref = oracle.step_window(grads, xw, np.float32(lib_stats["alpha"]), np.float32(lib_stats["c"]),
                             step=step, seed=seed, j0=j0, clip_limit=clip_limit,
                             payload_dtype=payload_dtype, rounding=rounding)
    if agg_dev is not None:
        assert np.array_equal(to_host(agg_dev[j0:j1]), ref["agg"]), f"aggregate mismatch in window {j0}:{j1}"
    assert np.array_equal(to_host(x_after_dev[j0:j1]).view(np.uint32), xw.view(np.uint32)), f"x mismatch in window {j0}:{j1}"
    return ref
