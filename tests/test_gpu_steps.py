"""GPU parity of whole IntSGD steps (exact first step, two-kernel and fused paths) with the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import LockStep, check_window, dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


FUSED_PIPELINED, FUSED_DIRECT, TWO_KERNEL = "fused-pipelined", "fused-direct", "two-kernel"


def _mode_and_path(which):
    return {FUSED_PIPELINED: (pkg.MODE_FUSED, 0), FUSED_DIRECT: (pkg.MODE_FUSED, 1), TWO_KERNEL: (pkg.MODE_TWO_KERNEL, 0)}[which]


@pytest.mark.parametrize("which", [FUSED_PIPELINED, FUSED_DIRECT, TWO_KERNEL])
@pytest.mark.parametrize("grad_dtype,payload_dtype", [(pkg.GRAD_F32, pkg.PAYLOAD_I32), (pkg.GRAD_F32, pkg.PAYLOAD_I8),
                                                      (pkg.GRAD_BF16, pkg.PAYLOAD_I8), (pkg.GRAD_BF16, pkg.PAYLOAD_I32)])
@pytest.mark.parametrize("rounding", [pkg.ROUND_RANDOM, pkg.ROUND_NEAREST, pkg.ROUND_RANDOM16, pkg.ROUND_RANDOM_COMPARE])
def test_multi_step_lockstep(which, grad_dtype, payload_dtype, rounding):
    """Several tiles and a ragged tail: d = 5 * 2^16 + 3 spans many blocks and leaves 3 coordinates."""
    n, d, eta = 6, 5 * (1 << 16) + 3, 0.1
    rng = np.random.default_rng(21)

    def grads():
        out = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        out[2][rng.integers(0, d, 50)] *= 300.0     # a few outliers: exercises clipping on the int8 wire
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    mode, path = _mode_and_path(which)
    ls = LockStep(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding, seed=99,
                  x0=rng.normal(0, 1, d).astype(np.float32), fused_path=path)
    try:
        ls.exact(grads(), eta)
        clipped = 0
        for k in range(5):
            st, ref = ls.step(grads(), eta, mode=mode)
            clipped += sum(st["clip_count"])
        if payload_dtype == pkg.PAYLOAD_I8:
            assert clipped > 0
    finally:
        ls.close()


@pytest.mark.parametrize("d", [(1 << 17) + 1, 4 * 2049 + 3, 2 * 4096, 9, 8])
@pytest.mark.parametrize("grad_dtype,payload_dtype,rounding", [
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM), (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM),
    (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM16),
    (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM16), (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM_COMPARE),
    (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_NEAREST)])
def test_two_kernel_payloads_match_the_oracle(d, grad_dtype, payload_dtype, rounding):
    """The payloads that the two-kernel step leaves in the caller's buffers are the oracle's encode of every worker
    (all workers in one launch of the pipelined encode kernel: whole tiles, a partial tile, the bf16 pair rule and
    the element-wise tail), with a few clipped and non-finite values planted."""
    n, eta, seed = 5, 0.2, 1234
    rng = np.random.default_rng(3)

    def grads():
        out = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        out[1][rng.integers(0, d, 4)] = [np.inf, -1e30, np.nan, 7.0]
        out[3][d - 1] = -np.inf
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    ls = LockStep(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding, seed=seed,
                  x0=rng.normal(0, 1, d).astype(np.float32))
    try:
        clean = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        ls.exact([synth.to_bf16_bits(g) for g in clean] if grad_dtype == pkg.GRAD_BF16 else clean, eta)
        for k in (1, 2):
            g = grads()
            st, ref = ls.step(g, eta, mode=pkg.MODE_TWO_KERNEL)
            for i in range(n):
                want, _, _ = oracle.encode(g[i], np.float32(st["alpha"]), worker=i, step=k, seed=seed, n=n,
                                           payload_dtype=payload_dtype, rounding=rounding)
                assert np.array_equal(ls.last_payloads[i], want), (k, i)
    finally:
        ls.close()


@pytest.mark.parametrize("which", [FUSED_PIPELINED, FUSED_DIRECT, TWO_KERNEL])
@pytest.mark.parametrize("grad_dtype,payload_dtype,rounding", [
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM),
    (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_NEAREST), (pkg.GRAD_BF16, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM),
    (pkg.GRAD_F32, pkg.PAYLOAD_I32, pkg.ROUND_RANDOM16), (pkg.GRAD_BF16, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM16),
    (pkg.GRAD_F32, pkg.PAYLOAD_I8, pkg.ROUND_RANDOM_COMPARE)])
def test_values_outside_the_fast_range_clip_and_count_exactly(which, grad_dtype, payload_dtype, rounding):
    """Huge, infinite and NaN gradients, and values between the fast-path range and the clip limit."""
    n, d, eta, seed = 5, 3 * 4096 + 9, 0.1, 77
    rng = np.random.default_rng(42)
    mode, path = _mode_and_path(which)
    x0 = rng.normal(0, 1, d).astype(np.float32)
    ls = LockStep(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding, seed=seed, x0=x0,
                  fused_path=path)

    def grads(plant):
        out = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        if plant:
            for i in range(n):
                idx = rng.integers(0, d, 40)
                out[i][idx[:8]] = [1e30, -1e30, np.inf, -np.inf, np.nan, 3e38, -3e38, 1e-40]
                out[i][idx[8:24]] *= 1e4       # far outside an int8 limit, inside the int32 one
                out[i][idx[24:]] = rng.choice([-1.0, 1.0], 16) * 10.0 ** rng.uniform(2, 7, 16)   # up to 2^27-ish
            out[0][d - 1], out[1][d - 2], out[2][d - 9] = np.nan, np.inf, -1e25    # in the ragged tail too
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    try:
        ls.exact(grads(False), eta)
        total_clip = total_nonf = 0
        for k in range(4):
            st, ref = ls.step(grads(True), eta, mode=mode)
            total_clip += sum(st["clip_count"])
            total_nonf += st["nonfinite"]
        assert total_clip > 0 and total_nonf > 0
    finally:
        ls.close()


@pytest.mark.parametrize("which", [FUSED_PIPELINED, FUSED_DIRECT, TWO_KERNEL])
@pytest.mark.parametrize("rounding", [pkg.ROUND_RANDOM, pkg.ROUND_RANDOM16, pkg.ROUND_RANDOM_COMPARE])
def test_values_next_to_integers_and_tiny_values(which, rounding):
    """Int(y) = floor(y + u) must be taken on the unrounded sum: scaled gradients a few ulps from an
    integer (both sides), exact integers, halves, and values down to the subnormals."""
    n, d, eta, seed = 4, 2 * 4096 + 5, 0.1, 5
    rng = np.random.default_rng(17)
    mode, path = _mode_and_path(which)
    ls = LockStep(n, d, rounding=rounding, seed=seed, x0=rng.normal(0, 1, d).astype(np.float32), fused_path=path)
    try:
        ls.exact([rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)], eta)
        for k in range(3):
            _, _, alpha, _ = oracle.scale(d, n, eta, ls.orc.beta, ls.orc.eps, ls.orc.r, ls.orc.dx2)
            grads = []
            for i in range(n):
                ints = rng.integers(-200, 201, d).astype(np.float64)
                off = rng.choice([0.0, 0.5, 2.0**-20, -(2.0**-20), 2.0**-16, -(2.0**-16), 2.0**-12, -(2.0**-12)], d)
                g = ((ints + off) / float(alpha)).astype(np.float32)
                for _ in range(2):      # and their fp32 neighbours
                    idx = rng.integers(0, d, d // 8)
                    g[idx] = np.nextafter(g[idx], np.float32(rng.choice([-1e9, 1e9])))
                tiny = rng.integers(0, d, d // 16)
                g[tiny] = (rng.choice([-1.0, 1.0], tiny.size) * 10.0 ** rng.uniform(-45, -6, tiny.size)).astype(np.float32)
                grads.append(g)
            st, ref = ls.step(grads, eta, mode=mode)
            assert sum(st["clip_count"]) == 0
    finally:
        ls.close()


@pytest.mark.parametrize("n,d", [(1, 1), (1, 5), (2, 3), (64, 1000), (3, 4), (16, 2), (2, 8), (3, 9), (5, 2049)])
def test_degenerate_shapes(n, d):
    rng = np.random.default_rng(n * 1000 + d)
    for mode, path in ((pkg.MODE_FUSED, 0), (pkg.MODE_FUSED, 1), (pkg.MODE_TWO_KERNEL, 0)):
        ls = LockStep(n, d, seed=1, x0=rng.normal(0, 1, d).astype(np.float32), fused_path=path)
        try:
            ls.exact([rng.normal(0, 1, d).astype(np.float32) for _ in range(n)], 0.1)
            for _ in range(3):
                ls.step([rng.normal(0, 1, d).astype(np.float32) for _ in range(n)], 0.1, mode=mode)
        finally:
            ls.close()


def test_fused_without_aggregate_output():
    n, d = 3, 70_001
    rng = np.random.default_rng(5)
    ls = LockStep(n, d, seed=2, x0=rng.normal(0, 1, d).astype(np.float32))
    try:
        ls.exact([rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)], 0.1)
        ls.step([rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)], 0.1, want_agg=False)
    finally:
        ls.close()


def test_results_do_not_depend_on_the_launch_shape_and_are_reproducible():
    n, d, seed = 4, (1 << 19) + 2, 31
    rng = np.random.default_rng(6)
    grads = [to_dev(rng.normal(0, 1e-2, d).astype(np.float32)) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    outs = []
    for threads, bps in [(256, 8), (256, 8), (128, 3), (512, 1), (32, 32)]:
        with pkg.IntSGD(n, d, seed=seed) as lib:
            lib.intsgd_set_launch(threads, bps)
            x = to_dev(x0.copy())
            agg = torch.zeros(d, dtype=torch.int32, device=dev())
            lib.intsgd_set_state(r=0.0, dx2=2e-3, alpha=0.0, c=0.0, step=1)
            lib.intsgd_step(grads, x, agg, eta_k=0.1, mode=pkg.MODE_FUSED)
            st = lib.intsgd_get_stats()
            outs.append((to_host(x), to_host(agg), st["dx2"], st["max_abs_agg"]))
    for o in outs[1:]:
        assert np.array_equal(o[0], outs[0][0]) and np.array_equal(o[1], outs[0][1]) and o[3] == outs[0][3]
        assert rel_close(o[2], outs[0][2], 1e-13)
    assert outs[0][2] == outs[1][2]     # same launch shape: bit-identical reduction


def test_checkpoint_resume_is_bit_exact():
    n, d, seed, eta = 3, 50_003, 17, 0.1
    rng = np.random.default_rng(7)
    steps = [[to_dev(rng.normal(0, 1e-2, d).astype(np.float32)) for _ in range(n)] for _ in range(10)]
    x0 = rng.normal(0, 1, d).astype(np.float32)

    def run(lib, x, lo, hi):
        for k in range(lo, hi):
            lib.intsgd_step(steps[k], x, None, eta_k=eta, mode=pkg.MODE_EXACT if k == 0 else pkg.MODE_FUSED)

    with pkg.IntSGD(n, d, seed=seed) as a:
        xa = to_dev(x0.copy())
        run(a, xa, 0, 10)
        sa = a.intsgd_get_stats()
    with pkg.IntSGD(n, d, seed=seed) as b:
        xb = to_dev(x0.copy())
        run(b, xb, 0, 5)
        saved = b.intsgd_get_state()
        x_saved = xb.clone()
    with pkg.IntSGD(n, d, seed=seed) as c:
        c.intsgd_set_state(r=saved.r, dx2=saved.dx2, alpha=saved.alpha, c=saved.c, step=saved.step)
        run(c, x_saved, 5, 10)
        sc = c.intsgd_get_stats()
    assert torch.equal(xa, x_saved)
    assert (sa["r"], sa["dx2"], sa["alpha"], sa["step"]) == (sc["r"], sc["dx2"], sc["alpha"], sc["step"])


def test_step_host_matches_the_device_path():
    n, d, seed, eta = 4, 300_001, 3, 0.1
    rng = np.random.default_rng(8)
    grads = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    with pkg.IntSGD(n, d, seed=seed) as a:
        xa = to_dev(x0.copy())
        agg_a = torch.zeros(d, dtype=torch.int32, device=dev())
        ga = [to_dev(g) for g in grads]
        a.intsgd_step(ga, xa, None, eta_k=eta, mode=pkg.MODE_EXACT)
        a.intsgd_step(ga, xa, agg_a, eta_k=eta, mode=pkg.MODE_FUSED)
        sa = a.intsgd_get_stats()
    with pkg.IntSGD(n, d, seed=seed) as b:
        hx = torch.from_numpy(x0.copy()).pin_memory()
        hg = [torch.from_numpy(g).pin_memory() for g in grads]
        hagg = torch.zeros(d, dtype=torch.int32).pin_memory()
        b.intsgd_step_host(hg, hx, None, eta_k=eta, mode=pkg.MODE_EXACT)
        b.intsgd_step_host(hg, hx, hagg, eta_k=eta, mode=pkg.MODE_FUSED)
        sb = b.intsgd_get_stats()
    assert np.array_equal(hx.numpy(), to_host(xa)) and np.array_equal(hagg.numpy(), to_host(agg_a))
    assert sa["dx2"] == sb["dx2"] and sa["alpha"] == sb["alpha"]


@pytest.mark.parametrize("grad_dtype,rounding", [(pkg.GRAD_F32, pkg.ROUND_RANDOM), (pkg.GRAD_BF16, pkg.ROUND_RANDOM16)])
def test_step_host_over_several_windows_matches_the_oracle(grad_dtype, rounding):
    """A vector longer than the host path's window (2^22 coordinates) is stepped window by window with
    the copies overlapped; integers and iterate must be those of the single-launch definition."""
    n, d, seed, eta = 2, 2 * (1 << 22) + 4101, 13, 0.1
    rng = np.random.default_rng(19)

    def grads():
        out = [rng.normal(0, 1e-2, d).astype(np.float32) for _ in range(n)]
        return [synth.to_bf16_bits(g) for g in out] if grad_dtype == pkg.GRAD_BF16 else out

    x0 = rng.normal(0, 1, d).astype(np.float32)
    orc = oracle.OracleIntSGD(n, d, seed=seed, rounding=rounding)
    x_ref = x0.copy()
    with pkg.IntSGD(n, d, grad_dtype=grad_dtype, seed=seed, rounding=rounding) as lib:
        hx = torch.from_numpy(x0.copy()).pin_memory()
        hagg = torch.zeros(d, dtype=torch.int32).pin_memory()
        g = grads()
        pin = lambda a: torch.from_numpy(a.view(np.int16).copy() if a.dtype == np.uint16 else a.copy()).pin_memory()
        hg = [pin(a) for a in g]
        lib.intsgd_step_host(hg, hx, None, eta_k=eta, mode=pkg.MODE_EXACT)
        ref = orc.exact_step(g, x_ref, eta)
        st = lib.intsgd_get_stats()
        assert np.array_equal(hx.numpy(), x_ref) and rel_close(st["dx2"], ref["dx2"]) and st["step"] == 1
        for k in range(2):
            g = grads()
            hg = [pin(a) for a in g]
            lib.intsgd_step_host(hg, hx, hagg, eta_k=eta, mode=pkg.MODE_FUSED)
            st = lib.intsgd_get_stats()
            ref = orc.int_step(g, x_ref, eta, alpha_c=(np.float32(st["alpha"]), np.float32(st["c"])))
            assert rel_close(st["alpha"], float(ref["alpha"])) and rel_close(st["r"], ref["r"])
            assert np.array_equal(hagg.numpy(), ref["agg"])
            assert np.array_equal(hx.numpy().view(np.uint32), x_ref.view(np.uint32))
            assert rel_close(st["dx2"], ref["dx2"]) and st["max_abs_agg"] == ref["max_abs_agg"]
            assert st["clip_count"] == ref["clip_count"] and st["step"] == k + 2


@pytest.mark.parametrize("blocks", [0, 3])
def test_steps_enqueued_back_to_back_equal_steps_run_one_by_one(blocks):
    """Without a host synchronisation between them the kernels of consecutive steps are chained by
    programmatic dependent launches (each may start while the one before is still running and waits before
    it reads the state); the results must be those of steps separated by synchronisations."""
    n, d, seed, eta, K = 4, (1 << 20) + 3, 23, 0.1, 25
    rng = np.random.default_rng(29)
    grads = [to_dev(rng.normal(0, 1e-2, d).astype(np.float32)) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    out = []
    for sync_every_step in (False, True):
        with pkg.IntSGD(n, d, seed=seed) as lib:
            if blocks:
                lib.intsgd_set_blocks([0, d // 3, d // 2 + 1, d])
            x = to_dev(x0.copy())
            agg = torch.zeros(d, dtype=torch.int32, device=dev())
            for k in range(K):
                lib.intsgd_step(grads, x, agg, eta_k=eta, mode=pkg.MODE_EXACT if k == 0 else pkg.MODE_FUSED)
                if sync_every_step:
                    lib.intsgd_get_stats()
            st = lib.intsgd_get_stats()
            out.append((to_host(x), to_host(agg), st))
    (xa, agga, sa), (xb, aggb, sb) = out
    assert np.array_equal(xa.view(np.uint32), xb.view(np.uint32)) and np.array_equal(agga, aggb)
    for key in ("r", "dx2", "alpha", "c", "step", "max_abs_agg", "clip_count"):
        assert sa[key] == sb[key], key
