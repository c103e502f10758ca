"""GPU parity of the individual C-ABI calls (scale, sqdiff, encode, aggregate) against the oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import REL, dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


def _grad(rng, d, scale, grad_dtype):
    g = rng.normal(0, scale, d).astype(np.float32)
    return synth.to_bf16_bits(g) if grad_dtype == pkg.GRAD_BF16 else g


def test_scale_is_bit_exact_given_the_same_inputs():
    rng = np.random.default_rng(0)
    for (d, n, beta, eps) in [(1 << 20, 4, 0.9, 1e-8), (4096, 16, 0.0, 0.0), (11_173_962, 16, 0.3, 1e-4), (1, 1, 0.6, 1e-6)]:
        with pkg.IntSGD(n, d, beta=beta, eps=eps) as lib:
            r_prev = 0.0
            for k in range(6):
                eta, dx2 = float(rng.uniform(0.01, 3)), float(rng.uniform(1e-9, 10))
                lib.intsgd_scale(eta, dx2)
                st = lib.intsgd_get_stats()
                r, a64, a32, c32 = oracle.scale(d, n, eta, beta, eps, r_prev, dx2)
                assert st["r"] == r and st["alpha"] == float(a32) and st["c"] == float(c32)
                r_prev = r


def test_scale_uses_the_stored_dx2_when_not_overridden():
    with pkg.IntSGD(2, 4, beta=0.0, eps=0.0) as lib:
        lib.intsgd_set_state(r=0.0, dx2=0.25, alpha=0.0, c=0.0, step=3)
        lib.intsgd_scale(0.5)
        st = lib.intsgd_get_stats()
        assert st["alpha"] == 1.0 and st["r"] == 0.25 and st["c"] == 0.25 and st["step"] == 3


def test_nonfinite_scale_is_reported_and_the_step_is_not_applied():
    d, n = 1024, 2
    g = [to_dev(np.ones(d, dtype=np.float32)) for _ in range(n)]
    x = to_dev(np.arange(d, dtype=np.float32))
    with pkg.IntSGD(n, d, beta=0.9, eps=0.0) as lib:
        lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_FUSED)    # r = 0 and eps = 0: alpha = inf
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_get_stats()
        assert e.value.code == pkg.ERR_SCALE_NONFINITE
        st = lib.intsgd_get_stats(allow_nonfinite=True)
        assert st["step"] == 0 and st["r"] == 0.0
        assert np.array_equal(to_host(x), np.arange(d, dtype=np.float32))
        # the context stays usable: an exact step, then a compressed one
        lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        lib.intsgd_step(g, x, None, eta_k=0.1, mode=pkg.MODE_FUSED)
        st = lib.intsgd_get_stats()
        assert st["status"] == pkg.OK and st["step"] == 2


@pytest.mark.parametrize("d", [1, 3, 4, 5, 1023, (1 << 16) + 2, 3 * (1 << 18) + 1])
def test_sqdiff(d):
    rng = np.random.default_rng(d)
    a = rng.normal(0, 1, d).astype(np.float32)
    b = (a + rng.normal(0, 1e-3, d)).astype(np.float32)
    with pkg.IntSGD(2, d) as lib:
        lib.intsgd_sqdiff(to_dev(a), to_dev(b))
        got = lib.intsgd_get_stats()["dx2"]
    assert rel_close(got, oracle.sqdiff(a, b), 1e-12)


@pytest.mark.parametrize("grad_dtype", [pkg.GRAD_F32, pkg.GRAD_BF16])
@pytest.mark.parametrize("payload_dtype", [pkg.PAYLOAD_I32, pkg.PAYLOAD_I8])
@pytest.mark.parametrize("rounding", [pkg.ROUND_RANDOM, pkg.ROUND_NEAREST, pkg.ROUND_RANDOM16, pkg.ROUND_RANDOM_COMPARE])
def test_encode_bit_exact(grad_dtype, payload_dtype, rounding):
    rng = np.random.default_rng(11)
    n, seed = 5, 0xDEADBEEFCAFE
    for d in [1, 2, 7, 4096, 3 * (1 << 17) + 3]:
        g = _grad(rng, d, 1.0, grad_dtype)
        if d > 100:   # plant values that clip, overflow and are not finite
            gf = synth.bf16_bits_to_f32(g) if grad_dtype == pkg.GRAD_BF16 else g
            gf = gf.copy()
            gf[5], gf[17], gf[70], gf[d - 1], gf[d - 2] = 1e30, -1e30, np.nan, np.inf, -np.inf
            gf[33], gf[34] = 3e38, -3e38
            g = synth.to_bf16_bits(gf) if grad_dtype == pkg.GRAD_BF16 else gf
        alpha = np.float32(47.3)
        pay_t = torch.int8 if payload_dtype == pkg.PAYLOAD_I8 else torch.int32
        with pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, rounding=rounding, seed=seed) as lib:
            lib.intsgd_set_state(r=0.0, dx2=0.0, alpha=1.0, c=1.0, step=9)
            lib.intsgd_scale(1.0, 1.0)   # opens the step (clears counters); alpha below is imposed
            out = torch.zeros(d, dtype=pay_t, device=dev())
            worker = 3
            lib.intsgd_encode(worker, to_dev(g), out, alpha_override=float(alpha))
            st = lib.intsgd_get_stats()
        want, clip, nonf = oracle.encode(g, alpha, worker=worker, step=9, seed=seed, n=n,
                                         payload_dtype=payload_dtype, rounding=rounding)
        assert np.array_equal(to_host(out), want)
        assert st["clip_count"][worker] == clip and sum(st["clip_count"]) == clip
        assert st["nonfinite"] == nonf


def test_encode_uses_the_state_alpha_and_step():
    d, n, seed = 10_001, 2, 5
    g = np.random.default_rng(1).normal(0, 1, d).astype(np.float32)
    with pkg.IntSGD(n, d, seed=seed) as lib:
        lib.intsgd_set_state(r=0.0, dx2=0.0, alpha=12.5, c=1.0, step=77)
        out = torch.zeros(d, dtype=torch.int32, device=dev())
        lib.intsgd_encode(1, to_dev(g), out)
        want, _, _ = oracle.encode(g, np.float32(12.5), worker=1, step=77, seed=seed, n=n)
        assert np.array_equal(to_host(out), want)


@pytest.mark.parametrize("payload_dtype", [pkg.PAYLOAD_I32, pkg.PAYLOAD_I8])
@pytest.mark.parametrize("d", [1, 6, 15, 16, 17, 4099, (1 << 18) + 13])
def test_aggregate_bit_exact(payload_dtype, d):
    rng = np.random.default_rng(d)
    n = 7
    lim = 127 if payload_dtype == pkg.PAYLOAD_I8 else 10_000
    np_t = np.int8 if payload_dtype == pkg.PAYLOAD_I8 else np.int32
    pays = [rng.integers(-lim, lim + 1, d).astype(np_t) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)
    c = np.float32(3.1e-4)
    x_ref = x0.copy()
    agg, dx2, ovf, mx = oracle.aggregate(pays, x_ref, c)
    for want_agg in (True, False):
        with pkg.IntSGD(n, d, payload_dtype=payload_dtype) as lib:
            lib.intsgd_set_state(r=0.0, dx2=0.0, alpha=1.0, c=float(c), step=4)
            x = to_dev(x0.copy())
            a = torch.zeros(d, dtype=torch.int32, device=dev()) if want_agg else None
            lib.intsgd_aggregate([to_dev(p) for p in pays], x, a)
            st = lib.intsgd_get_stats()
        if want_agg:
            assert np.array_equal(to_host(a), agg)
        assert np.array_equal(to_host(x).view(np.uint32), x_ref.view(np.uint32))
        assert rel_close(st["dx2"], dx2, 1e-12)
        assert st["agg_overflow"] == ovf and st["max_abs_agg"] == mx and st["step"] == 5


def test_unaligned_pointers_take_the_elementwise_path():
    rng = np.random.default_rng(2)
    n, d, seed = 3, 10_007, 8
    for grad_dtype, pay_dtype in [(pkg.GRAD_F32, pkg.PAYLOAD_I32), (pkg.GRAD_BF16, pkg.PAYLOAD_I8)]:
        grads = [_grad(rng, d, 1e-2, grad_dtype) for _ in range(n)]
        x0 = rng.normal(0, 1, d).astype(np.float32)
        # views that start one element into a larger buffer: aligned to the element, not to 16 bytes
        def off(a):
            t = to_dev(np.concatenate([a[:1], a]))
            return t[1:]
        g_dev = [off(g) for g in grads]
        x_dev = off(x0)
        agg_dev = torch.zeros(d + 1, dtype=torch.int32, device=dev())[1:]
        pay_t = torch.int8 if pay_dtype == pkg.PAYLOAD_I8 else torch.int32
        scratch = [torch.zeros(d + 1, dtype=pay_t, device=dev())[1:] for _ in range(n)]
        assert x_dev.data_ptr() % 16 != 0
        for mode in (pkg.MODE_FUSED, pkg.MODE_TWO_KERNEL):
            x_dev.copy_(torch.from_numpy(x0))
            with pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=pay_dtype, seed=seed) as lib:
                lib.intsgd_set_state(r=0.0, dx2=1e-3, alpha=0.0, c=0.0, step=1)
                lib.intsgd_step(g_dev, x_dev, agg_dev, eta_k=0.1, mode=mode, payload_scratch=scratch)
                st = lib.intsgd_get_stats()
            x_ref = x0.copy()
            ref = oracle.step_window(grads, x_ref, np.float32(st["alpha"]), np.float32(st["c"]), step=1, seed=seed,
                                     payload_dtype=pay_dtype)
            assert np.array_equal(to_host(agg_dev), ref["agg"])
            assert np.array_equal(to_host(x_dev), x_ref)
            assert st["clip_count"] == ref["clip_count"] and st["agg_overflow"] == ref["agg_overflow"]


def test_misaligned_to_element_size_is_an_error_not_a_fault():
    d = 64
    with pkg.IntSGD(1, d) as lib:
        buf = torch.zeros(d + 4, dtype=torch.float32, device=dev())
        x = torch.zeros(d, dtype=torch.float32, device=dev())
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_step([buf.data_ptr() + 2], x, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        assert e.value.code == pkg.ERR_ALIGN
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_step([buf], None, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        assert e.value.code == pkg.ERR_INVALID_ARG
        for bad_eta in (0.0, -1.0, math.inf, math.nan):
            with pytest.raises(pkg.IntSGDError) as e:
                lib.intsgd_step([buf], x, None, eta_k=bad_eta, mode=pkg.MODE_FUSED)
            assert e.value.code == pkg.ERR_INVALID_ARG
        with pytest.raises(pkg.IntSGDError):
            lib.intsgd_encode(1, buf, torch.zeros(d, dtype=torch.int32, device=dev()))   # worker out of range
        with pytest.raises(pkg.IntSGDError):
            lib.intsgd_step([buf], x, None, eta_k=0.1, mode=pkg.MODE_TWO_KERNEL)   # no scratch
        assert "scratch" in lib.intsgd_last_error()


def test_an_expired_wait_is_reported_and_the_context_stays_usable():
    """The failure path without a GPU fault: the library's bounded wait runs out on a barrier that nothing
    completes; the status is INTSGD_ERR_TIMEOUT until the state is set again, and the context then steps
    exactly like a fresh one."""
    n, d, eta, seed = 3, 5000, 0.1, 11
    rng = np.random.default_rng(21)
    grads = [to_dev(rng.normal(0, 1e-2, d).astype(np.float32)) for _ in range(n)]
    x0 = rng.normal(0, 1, d).astype(np.float32)

    def two_steps(lib):
        x, agg = to_dev(x0.copy()), torch.zeros(d, dtype=torch.int32, device=dev())
        lib.intsgd_step(grads, x, None, eta_k=eta, mode=pkg.MODE_EXACT)
        lib.intsgd_step(grads, x, agg, eta_k=eta)
        return to_host(x), to_host(agg), lib.intsgd_get_stats()

    with pkg.IntSGD(n, d, seed=seed) as lib:
        lib.intsgd_selftest_wait_expiry()
        for _ in range(2):   # sticky
            with pytest.raises(pkg.IntSGDError) as err:
                lib.intsgd_get_stats()
            assert err.value.code == pkg.ERR_TIMEOUT
        # the state block was read although the call reports the expiry: intsgd_get_state fills its output
        import ctypes
        from paper_2102_08374_b200 import binding
        lib.intsgd_set_state(r=0.25, dx2=0.5, alpha=3.0, c=0.125, step=7)      # clears the flag ...
        lib.intsgd_selftest_wait_expiry()                                       # ... and this sets it again
        raw = binding.State(r=-1.0, dx2=-1.0, alpha=-1.0, c=-1.0, step=99, status=55)
        assert lib._lib.intsgd_get_state(lib._ctx, ctypes.byref(raw)) == pkg.ERR_TIMEOUT
        assert (raw.r, raw.dx2, raw.alpha, raw.c, raw.step, raw.status) == (0.25, 0.5, 3.0, 0.125, 7, pkg.OK)
        lib.intsgd_set_state(r=0.0, dx2=0.0, alpha=0.0, c=0.0, step=0)
        assert lib.intsgd_get_stats()["step"] == 0
        x_a, agg_a, st_a = two_steps(lib)
    with pkg.IntSGD(n, d, seed=seed) as fresh:
        x_b, agg_b, st_b = two_steps(fresh)
    assert np.array_equal(x_a.view(np.uint32), x_b.view(np.uint32)) and np.array_equal(agg_a, agg_b)
    assert st_a["alpha"] == st_b["alpha"] and st_a["dx2"] == st_b["dx2"] and st_a["step"] == st_b["step"] == 2


def test_philox_rate_diagnostic_runs_and_checks_its_arguments():
    """The register-only Philox kernel behind the benchmark's arithmetic ceiling: it reports how many blocks a launch
    computes, touches no vector and no state, and refuses arguments outside its documented set."""
    with pkg.IntSGD(2, 64) as lib:
        before = lib.intsgd_get_stats()
        sms = torch.cuda.get_device_properties(dev()).multi_processor_count
        for extra in (0, 16, 32):
            assert lib.intsgd_selftest_philox_rate(64, extra) == sms * 512 * 64
        assert lib.intsgd_selftest_philox_rate(7) == sms * 512 * 6          # rounded down to even
        for bad in (dict(blocks_per_thread=1), dict(blocks_per_thread=(1 << 24) + 2), dict(blocks_per_thread=64, extra_ops_per_block=5)):
            with pytest.raises(pkg.IntSGDError) as e:
                lib.intsgd_selftest_philox_rate(**bad)
            assert e.value.code == pkg.ERR_INVALID_ARG
        after = lib.intsgd_get_stats()
        assert {k: before[k] for k in ("r", "dx2", "alpha", "c", "step")} == {k: after[k] for k in ("r", "dx2", "alpha", "c", "step")}


def test_a_failed_staging_allocation_of_the_host_step_leaks_nothing():
    """intsgd_step_host allocates its device staging on first use, all or nothing: when the buffers cannot be had
    (here 2 x 512 GiB, more than the GPU holds) the call fails with INTSGD_ERR_CUDA before it reads a single host
    byte, what the attempt had obtained is released, and a second attempt behaves the same."""
    import ctypes
    n, d = 2, 1 << 37
    with pkg.IntSGD(n, d) as lib:
        host = np.zeros(16, dtype=np.float32)                     # never read: the allocation fails first
        ptrs = (ctypes.c_void_p * n)(*[host.ctypes.data] * n)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for _ in range(2):
            rc = lib._lib.intsgd_step_host(lib._ctx, ptrs, host.ctypes.data, None, 0.1, pkg.MODE_EXACT, None)
            assert rc == pkg.ERR_CUDA and "staging" in lib.intsgd_last_error()
            free1, _ = torch.cuda.mem_get_info()
            assert abs(free1 - free0) < (64 << 20)                # nothing of the failed attempt is kept
