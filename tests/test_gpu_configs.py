"""GPU parity on the five benchmark configurations (synthetic stand-ins for the paper's workloads).

Small vectors are compared in full every step; for the large ones the oracle recomputes sampled
coordinate windows (the random stream is indexed by absolute coordinate) and the squared step
length is checked against an fp64 reduction of the library's own iterates.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import LockStep, check_window, dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


def _dx2_fp64(x_after, x_before):
    return float(((x_after - x_before).double() ** 2).sum().item())


def _clipped(g, alpha_t, limit):
    """Coordinates of one worker whose scaled value leaves the clip range: the counter's definition, evaluated
    with one separately rounded fp32 multiply on the device."""
    return int((~((g * alpha_t).abs() <= limit)).sum().item())


class ScalarChain:
    """The oracle's scalar recursion (r_k, alpha_k, c_k) driven by the measured step lengths."""

    def __init__(self, n, d, beta=0.9, eps=1e-8):
        self.n, self.d, self.beta, self.eps, self.r = n, d, beta, eps, 0.0

    def advance(self, eta, dx2, st):
        self.r, a64, a32, c32 = oracle.scale(self.d, self.n, eta, self.beta, self.eps, self.r, dx2)
        assert rel_close(st["r"], self.r), (st["r"], self.r)
        assert rel_close(st["alpha"], float(a32)) and rel_close(st["c"], float(c32))


def test_config1_operator_check():
    w = synth.operator_check()
    n, d, eta = w["n"], w["d"], w["eta"]
    seed = 0
    for mode in (pkg.MODE_FUSED, pkg.MODE_TWO_KERNEL):
        with pkg.IntSGD(n, d, beta=w["beta"], eps=w["eps"], seed=seed) as lib:
            x = to_dev(w["x0"].copy())
            agg = torch.zeros(d, dtype=torch.int32, device=dev())
            scratch = [torch.zeros(d, dtype=torch.int32, device=dev()) for _ in range(n)]
            lib.intsgd_sqdiff(x, to_dev(w["x_prev"]))
            dx2_gpu = lib.intsgd_get_stats()["dx2"]
            dx2_ref = oracle.sqdiff(w["x0"], w["x_prev"])
            assert rel_close(dx2_gpu, dx2_ref, 1e-12)
            lib.intsgd_step([to_dev(g) for g in w["grads"]], x, agg, eta_k=eta, mode=mode, payload_scratch=scratch)
            st = lib.intsgd_get_stats()
        r, a64, a32, c32 = oracle.scale(d, n, eta, w["beta"], w["eps"], 0.0, dx2_ref)
        assert rel_close(st["r"], r) and rel_close(st["alpha"], float(a32))
        assert 0.09 < st["r"] < 0.12 and 100 < st["alpha"] < 125      # r ~ 0.105, alpha ~ 112
        x_ref = w["x0"].copy()
        ref = oracle.step_window(w["grads"], x_ref, np.float32(st["alpha"]), np.float32(st["c"]), step=0, seed=seed)
        assert np.array_equal(to_host(agg), ref["agg"])
        assert np.array_equal(to_host(x).view(np.uint32), x_ref.view(np.uint32))
        assert rel_close(st["dx2"], ref["dx2"])
        assert st["clip_count"] == ref["clip_count"] == [0] * n
        assert st["max_abs_agg"] == ref["max_abs_agg"]
        if mode == pkg.MODE_TWO_KERNEL:
            for i in range(n):
                want, _, _ = oracle.encode(w["grads"][i], np.float32(st["alpha"]), worker=i, step=0, seed=seed, n=n)
                assert np.array_equal(to_host(scratch[i]), want)


def test_config2_logistic_regression_500_steps():
    n, d, eta, steps, seed = 16, 4096, 0.5, 500, 2
    prob = synth.LogisticProblem(n=n, d=d, device=dev())
    ls = LockStep(n, d, seed=seed, x0=np.zeros(d, dtype=np.float32))
    try:
        max_int = []
        for k in range(steps):
            g_dev = prob.gradients(ls.x_dev)
            grads = [to_host(g) for g in g_dev]
            if k == 0:
                ls.exact(grads, eta)
                continue
            mode = pkg.MODE_FUSED if k % 2 else pkg.MODE_TWO_KERNEL
            st, ref = ls.step(grads, eta, mode=mode, g_dev=g_dev)
            max_int.append(st["max_abs_agg"])
        # every step was compared in full; the largest aggregated integer (the quantity plotted in
        # Appendix C.5) stays far inside the int32 wire type on this stand-in problem
        assert 0 < max(max_int) < 2**27
    finally:
        ls.close()


def test_heterogeneous_workers_drive_the_integers_past_2_23_and_into_the_clip():
    """Appendix A.2 / C.5 of the paper: on heterogeneous data the local gradients do not vanish at the optimum, so
    as the iterates converge alpha_k grows and the transmitted integers grow with it.  A small, strongly
    heterogeneous logistic regression (64 workers of 8 samples) is driven, in lock step with the oracle on the
    whole vector every step, through three regimes: values beyond the pipelined kernel's float-accumulation range
    (redone exactly), |alpha g| >= 2^23 (no fractional bits: Int is deterministic), and the int32 clip limit
    floor((2^31 - 1) / n) (counted, after which the large step makes alpha collapse and regrow)."""
    n, m, d, eta, steps, seed = 64, 8, 256, 0.5, 300, 2
    prob = synth.LogisticProblem(n=n, m=m, d=d, lam=0.1, device=dev())
    limit = oracle.limit_as_float(oracle.default_clip_limit(n, pkg.PAYLOAD_I32))
    paths = [(pkg.MODE_FUSED, 0), (pkg.MODE_TWO_KERNEL, 0), (pkg.MODE_FUSED, 1)]
    ls = LockStep(n, d, seed=seed, beta=0.5, x0=np.zeros(d, dtype=np.float32))
    try:
        beyond_fast = beyond_23 = clipped_steps = 0
        max_int = 0
        for k in range(steps):
            g_dev = prob.gradients(ls.x_dev)
            grads = [to_host(g) for g in g_dev]
            if k == 0:
                ls.exact(grads, eta)
                continue
            mode, path = paths[k % 3]
            ls.lib.intsgd_set_fused_path(path)
            st, ref = ls.step(grads, eta, mode=mode, g_dev=g_dev)
            ymax = st["alpha"] * max(float(np.abs(g).max()) for g in grads)
            beyond_fast += ymax > (1 << 24) / n
            beyond_23 += ymax >= 2.0 ** 23
            clipped_steps += sum(st["clip_count"]) > 0
            max_int = max(max_int, st["max_abs_agg"])
            assert ymax <= limit or sum(st["clip_count"]) > 0
        assert beyond_fast > 20 and beyond_23 > 3 and clipped_steps >= 1
        assert max_int > 1 << 20        # the clipped step's aggregate is no longer a sum of cancelling integers
    finally:
        ls.close()


def test_config3_resnet18_shaped_200_steps():
    n, d, eta, steps, seed, pool = 16, synth.RESNET18_D, 0.1, 200, 3, 4
    assert d % 4 == 2
    sets = [[to_dev(synth.resnet18_gradient(i, p)) for i in range(n)] for p in range(pool)]
    x = to_dev(synth.iterate(d, seed=33))
    agg = torch.zeros(d, dtype=torch.int32, device=dev())
    scratch = [torch.empty(d, dtype=torch.int32, device=dev()) for _ in range(n)]
    chain = ScalarChain(n, d)
    # windows: start, the ragged end, one that crosses several small (batch-norm) segments
    windows = [(0, 1 << 15), (d - 30_001, d), (1728 + 64, 1728 + 64 + 40_000), (5_000_001, 5_000_001 + (1 << 15))]
    full_steps = {1, 2, 150}      # the whole vector, counters included: two early steps and a late one
    sampled = {1, 2, 3, 50, 101, 150, 199}
    with pkg.IntSGD(n, d, seed=seed) as lib:
        dx2_prev = None
        for k in range(steps):
            g = sets[k % pool]
            x_before = x.clone() if (k in sampled or k == 0) else None
            mode = pkg.MODE_EXACT if k == 0 else (pkg.MODE_TWO_KERNEL if k % 10 == 5 else pkg.MODE_FUSED)
            lib.intsgd_step(g, x, agg, eta_k=eta, mode=mode, payload_scratch=scratch)
            st = lib.intsgd_get_stats()
            if k > 0:
                chain.advance(eta, dx2_prev, st)
            dx2_prev = st["dx2"]
            if k == 0:
                x_ref = to_host(x_before)
                ref_dx2 = oracle.exact_step([to_host(t) for t in g], x_ref, eta)
                assert np.array_equal(to_host(x), x_ref) and rel_close(st["dx2"], ref_dx2)
            elif k in full_steps:
                x_ref = to_host(x_before)
                ref = oracle.step_window([to_host(t) for t in g], x_ref, np.float32(st["alpha"]), np.float32(st["c"]),
                                         step=k, seed=seed)
                assert np.array_equal(to_host(agg), ref["agg"])
                assert np.array_equal(to_host(x).view(np.uint32), x_ref.view(np.uint32))
                assert rel_close(st["dx2"], ref["dx2"])
                assert st["clip_count"] == ref["clip_count"] and st["max_abs_agg"] == ref["max_abs_agg"]
                assert st["nonfinite"] == ref["nonfinite"] and st["agg_overflow"] == ref["agg_overflow"]
            elif k in sampled:
                for (j0, j1) in windows:
                    check_window(st, g, x_before, x, agg, j0, j1, step=k, seed=seed, n=n)
                assert rel_close(st["dx2"], _dx2_fp64(x, x_before))
                assert st["max_abs_agg"] == int(agg.abs().max().item())
        assert st["step"] == steps


def test_config4_lstm_shaped_bf16_int8_200_steps():
    n, d, steps, seed, pool = 8, 1 << 25, 200, 4, 2
    sets = [[to_dev(synth.lstm_gradient_bf16(i, d, p)) for i in range(n)] for p in range(pool)]
    x = to_dev(synth.iterate(d, seed=44))
    agg = torch.zeros(d, dtype=torch.int32, device=dev())
    scratch = [torch.empty(d, dtype=torch.int8, device=dev()) for _ in range(n)]
    chain = ScalarChain(n, d)
    k_emb = (d * 2) // 5
    windows = [(0, 1 << 15), (d - (1 << 15), d), (k_emb - 20_000, k_emb + 20_000), (17_000_003, 17_000_003 + (1 << 15))]
    sampled = {2, 3, 60, 99, 100, 101, 160, 199}
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16, payload_dtype=pkg.PAYLOAD_I8, seed=seed) as lib:
        dx2_prev = None
        saw_clip = saw_overflow = False
        for k in range(steps):
            g, eta = sets[k % pool], synth.lstm_eta(k)
            x_before = x.clone() if (k in sampled or k <= 1) else None
            mode = pkg.MODE_EXACT if k == 0 else (pkg.MODE_TWO_KERNEL if k % 10 == 3 else pkg.MODE_FUSED)
            lib.intsgd_step(g, x, agg, eta_k=eta, mode=mode, payload_scratch=scratch)
            st = lib.intsgd_get_stats()
            if k > 0:
                chain.advance(eta, dx2_prev, st)
                saw_clip |= sum(st["clip_count"]) > 0
                saw_overflow |= st["agg_overflow"] > 0
            dx2_prev = st["dx2"]
            if k == 0:
                x_ref = to_host(x_before)
                ref_dx2 = oracle.exact_step([to_host(t) for t in g], x_ref, eta)
                assert np.array_equal(to_host(x), x_ref) and rel_close(st["dx2"], ref_dx2)
            elif k in (1, 101):   # the whole vector, counters included: at the start and right after eta drops (alpha jumps)
                x_ref = to_host(x_before)
                ref = oracle.step_window([to_host(t) for t in g], x_ref, np.float32(st["alpha"]), np.float32(st["c"]),
                                         step=k, seed=seed, payload_dtype=pkg.PAYLOAD_I8)
                assert np.array_equal(to_host(agg), ref["agg"])
                assert np.array_equal(to_host(x).view(np.uint32), x_ref.view(np.uint32))
                assert rel_close(st["dx2"], ref["dx2"])
                assert st["clip_count"] == ref["clip_count"] and st["nonfinite"] == ref["nonfinite"]
                assert st["agg_overflow"] == ref["agg_overflow"] and st["max_abs_agg"] == ref["max_abs_agg"]
            elif k in sampled:
                for (j0, j1) in windows:
                    check_window(st, g, x_before, x, agg, j0, j1, step=k, seed=seed, n=n, payload_dtype=pkg.PAYLOAD_I8)
                assert rel_close(st["dx2"], _dx2_fp64(x, x_before))
                assert st["max_abs_agg"] == int(agg.abs().max().item())
                assert st["agg_overflow"] == int((agg.abs() > 127).sum().item())
                if mode == pkg.MODE_TWO_KERNEL:
                    for i in (0, n - 1):
                        j0, j1 = windows[2]
                        want, _, _ = oracle.encode(to_host(g[i][j0:j1]), np.float32(st["alpha"]), worker=i, step=k,
                                                   seed=seed, n=n, payload_dtype=pkg.PAYLOAD_I8, j0=j0)
                        assert np.array_equal(to_host(scratch[i][j0:j1]), want)
        assert saw_clip     # the heavy-tailed embedding part reaches the +-127 limit


SWEEP = [(22, 2), (22, 8), (22, 16), (24, 2), (24, 8), (24, 16), (26, 2), (26, 8), (26, 16), (28, 2), (28, 8), (28, 16)]


@pytest.mark.parametrize("log2d,n", SWEEP)
def test_config5_bucket_sweep(log2d, n):
    """d in {2^22..2^28} x n in {2, 8, 16}, int32 and int8 wire, two-kernel and fused, 50 steps each,
    in the launch shape the benchmark times (the library default)."""
    d, eta, steps = 1 << log2d, 0.1, 50
    grads = synth.bucket_gradients_device(n, d, dev())
    x0 = synth.iterate_device(d, dev())
    agg = torch.zeros(d, dtype=torch.int32, device=dev())
    wsize = 1 << 15
    rng = np.random.default_rng(log2d * 100 + n)
    windows = [(0, wsize), (d - wsize, d)] + [(int(j), int(j) + wsize) for j in rng.integers(0, d - wsize, 2)]
    sampled = {1, 25, 49}
    for payload_dtype in (pkg.PAYLOAD_I32, pkg.PAYLOAD_I8):
        pay_t = torch.int8 if payload_dtype == pkg.PAYLOAD_I8 else torch.int32
        scratch = [torch.empty(d, dtype=pay_t, device=dev()) for _ in range(n)]
        for mode in (pkg.MODE_FUSED, pkg.MODE_TWO_KERNEL):
            seed = 5000 + log2d
            x = x0.clone()
            chain = ScalarChain(n, d)
            with pkg.IntSGD(n, d, payload_dtype=payload_dtype, seed=seed) as lib:
                dx2_prev = None
                for k in range(steps):
                    x_before = x.clone() if k in sampled else None
                    lib.intsgd_step(grads, x, agg, eta_k=eta, mode=pkg.MODE_EXACT if k == 0 else mode,
                                    payload_scratch=scratch)
                    if k in sampled or k == 0 or k - 1 in sampled:
                        st = lib.intsgd_get_stats()
                    if k in sampled:
                        if k == 1:
                            chain.r = 0.0
                            chain.advance(eta, dx2_prev, st)
                        limit = oracle.limit_as_float(oracle.default_clip_limit(n, payload_dtype))
                        alpha_t = torch.tensor(st["alpha"], dtype=torch.float32, device=dev())
                        for (j0, j1) in windows:
                            ref = check_window(st, grads, x_before, x, agg, j0, j1, step=k, seed=seed, n=n,
                                               payload_dtype=payload_dtype)
                            # the oracle's counters on the window against the counter's definition, !(|fl32(alpha g)| <= Lf)
                            assert ref["clip_count"] == [_clipped(g[j0:j1], alpha_t, limit) for g in grads]
                            assert ref["max_abs_agg"] == int(agg[j0:j1].abs().max().item())
                        assert rel_close(st["dx2"], _dx2_fp64(x, x_before))
                        assert st["max_abs_agg"] == int(agg.abs().max().item())
                        # the library's counters on the whole vector against the same definition
                        assert st["clip_count"] == [_clipped(g, alpha_t, limit) for g in grads]
                        assert st["nonfinite"] == 0
                        assert st["agg_overflow"] == (int((agg.abs() > 127).sum().item()) if payload_dtype == pkg.PAYLOAD_I8 else 0)
                    if k == 0:
                        dx2_prev = st["dx2"]
                assert lib.intsgd_get_stats()["step"] == steps
        del scratch
