"""ctypes binding of the IntSGD CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

The arithmetic lives in ``intsgd_oracle.cpp`` (plain single-threaded C++, fp32 operations
rounded one by one, own Philox4x32-10).  This module compiles it with g++ on first use, exposes
its functions and strings them together in the order of Algorithm 1 of the IntSGD paper
(``OracleIntSGD``).  Only tests, the smoke check and the benchmark's CPU-baseline leg import it;
it imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "intsgd_oracle.cpp"
_LIB = _HERE / "liboracle_intsgd.so"

GRAD_F32, GRAD_BF16 = 0, 1
PAYLOAD_I32, PAYLOAD_I8 = 0, 1
ROUND_RANDOM, ROUND_NEAREST, ROUND_RANDOM16, ROUND_RANDOM_COMPARE = 0, 1, 2, 3
INT32_MAX = 2**31 - 1


def build(force: bool = False) -> Path:
    """Compile the oracle (g++, no FMA contraction, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-Wall",
             "-shared", "-fPIC", "-o", str(tmp), str(_SRC)], check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _declare(L: C.CDLL) -> C.CDLL:
    """Attach argument and result types to the oracle's entry points."""
    u32p, f32p, i32p = C.POINTER(C.c_uint32), C.POINTER(C.c_float), C.POINTER(C.c_int32)
    f64p, u64p = C.POINTER(C.c_double), C.POINTER(C.c_uint64)
    L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
    L.orc_philox4x32_10.restype = None
    L.orc_draw_word.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
    L.orc_draw_word.restype = C.c_uint32
    L.orc_uniform_from_word.argtypes = [C.c_uint32]
    L.orc_uniform_from_word.restype = C.c_float
    L.orc_draw_uniform16.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint64]
    L.orc_draw_uniform16.restype = C.c_float
    L.orc_int_round.argtypes = [C.c_float, C.c_float]
    L.orc_int_round.restype = C.c_int32
    L.orc_int_round_nearest.argtypes = [C.c_float]
    L.orc_int_round_nearest.restype = C.c_int32
    L.orc_int_round_compare.argtypes = [C.c_float, C.c_float]
    L.orc_int_round_compare.restype = C.c_int32
    L.orc_uniform24_from_word.argtypes = [C.c_uint32]
    L.orc_uniform24_from_word.restype = C.c_float
    L.orc_limit_as_float.argtypes = [C.c_int64]
    L.orc_limit_as_float.restype = C.c_float
    L.orc_scale.argtypes = [C.c_int64, C.c_int32, C.c_double, C.c_double, C.c_double,
                            C.c_double, C.c_double, f64p, f64p, f32p, f32p]
    L.orc_scale.restype = None
    L.orc_scale_block.argtypes = [C.c_int64, C.c_int64, C.c_int32, C.c_double, C.c_double,
                                  C.c_double, C.c_double, C.c_double, f64p, f64p, f32p, f32p]
    L.orc_scale_block.restype = None
    L.orc_encode.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_float, C.c_int64,
                             C.c_int, C.c_int, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p,
                             C.c_void_p, u64p, u64p]
    L.orc_encode.restype = None
    L.orc_aggregate.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int32, C.c_int64,
                                C.c_float, C.c_void_p, C.c_void_p, f64p, u64p, i32p]
    L.orc_aggregate.restype = None
    L.orc_exact_step.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int32, C.c_int64,
                                 C.c_double, C.c_void_p, f64p]
    L.orc_exact_step.restype = None
    L.orc_sqdiff.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
    L.orc_sqdiff.restype = C.c_double
    L.orc_step_window.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int32, C.c_int64,
                                  C.c_int64, C.c_float, C.c_float, C.c_int64, C.c_int, C.c_int,
                                  C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                  f64p, u64p, u64p, u64p, i32p]
    L.orc_step_window.restype = None
    L.orc_diana_step_window.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_int32, C.c_int64, C.c_int64,
                                        C.c_float, C.c_float, C.c_float, C.c_float, C.c_int64, C.c_int,
                                        C.c_int, C.c_uint64, C.c_uint32, C.POINTER(C.c_void_p), C.c_void_p,
                                        C.c_void_p, C.c_void_p, f64p, u64p, u64p, u64p, i32p]
    L.orc_diana_step_window.restype = None
    L.orc_heuristic_scale.argtypes = [C.c_float, C.c_int32, C.c_int32, C.c_double, i32p, f32p, f32p]
    L.orc_heuristic_scale.restype = C.c_int
    return L


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = _declare(C.CDLL(str(build())))
    return _lib


# --------------------------------------------------------------------------- small helpers
def _ptr(a: np.ndarray | None) -> C.c_void_p:
    return C.c_void_p(None) if a is None else C.c_void_p(a.ctypes.data)


def _grad_dtype(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return GRAD_F32
    if a.dtype == np.uint16:  # bf16 bit patterns
        return GRAD_BF16
    raise TypeError(f"gradient must be float32 or uint16 (bf16 bits), got {a.dtype}")


def _ptr_array(arrs) -> C.Array:
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def default_clip_limit(n: int, payload_dtype: int) -> int:
    """int8 wire: 127.  int32 wire: floor((2^31 - 1) / n), so the sum of n payloads fits."""
    return 127 if payload_dtype == PAYLOAD_I8 else INT32_MAX // n


def philox4x32_10(ctr, key) -> tuple[int, int, int, int]:
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return tuple(int(v) for v in o)


def draw_word(seed: int, step: int, worker: int, j: int) -> int:
    return int(lib().orc_draw_word(seed, step, worker, j))


def draw_uniform16(seed: int, step: int, worker: int, j: int) -> float:
    return float(lib().orc_draw_uniform16(seed, step, worker, j))


def uniform_from_word(w: int) -> float:
    return float(lib().orc_uniform_from_word(w))


def int_round(y: float, u: float) -> int:
    return int(lib().orc_int_round(y, u))


def int_round_compare(y: float, u: float) -> int:
    return int(lib().orc_int_round_compare(y, u))


def uniform24_from_word(w: int) -> float:
    return float(lib().orc_uniform24_from_word(w))


def int_round_nearest(y: float) -> int:
    return int(lib().orc_int_round_nearest(y))


def limit_as_float(L: int) -> float:
    return float(lib().orc_limit_as_float(L))


def scale(d, n, eta, beta, eps, r_prev, dx2):
    """(r_k, alpha_k in fp64, alpha_k rounded to fp32, c_k = eta/(n alpha_k) in fp32)."""
    r, a64 = C.c_double(), C.c_double()
    a32, c32 = C.c_float(), C.c_float()
    lib().orc_scale(d, n, eta, beta, eps, r_prev, dx2, C.byref(r), C.byref(a64), C.byref(a32),
                    C.byref(c32))
    return r.value, a64.value, np.float32(a32.value), np.float32(c32.value)


def scale_block(d, d_l, n, eta, beta, eps, r_prev, dx2):
    r, a64 = C.c_double(), C.c_double()
    a32, c32 = C.c_float(), C.c_float()
    lib().orc_scale_block(d, d_l, n, eta, beta, eps, r_prev, dx2, C.byref(r), C.byref(a64),
                          C.byref(a32), C.byref(c32))
    return r.value, a64.value, np.float32(a32.value), np.float32(c32.value)


def encode(grad, alpha, *, worker, step, seed, n=None, clip_limit=None,
           payload_dtype=PAYLOAD_I32, rounding=ROUND_RANDOM, j0=0, u_inject=None):
    """Int(alpha * grad) for one worker over coordinates [j0, j0 + len(grad)).

    Returns (payload, clip_count, nonfinite_count)."""
    grad = np.ascontiguousarray(grad)
    if clip_limit is None:
        clip_limit = default_clip_limit(n, payload_dtype)
    out = np.empty(grad.shape[0], dtype=np.int8 if payload_dtype == PAYLOAD_I8 else np.int32)
    clip, nonf = C.c_uint64(0), C.c_uint64(0)
    if u_inject is not None:
        u_inject = np.ascontiguousarray(u_inject, dtype=np.float32)
    lib().orc_encode(_ptr(grad), _grad_dtype(grad), j0, grad.shape[0], float(alpha),
                     int(clip_limit), payload_dtype, rounding, seed, step, worker,
                     _ptr(u_inject), _ptr(out), C.byref(clip), C.byref(nonf))
    return out, clip.value, nonf.value


def aggregate(payloads, x, c, *, want_agg=True):
    """Sum the payloads, decode with c = eta/(n alpha), update x in place.

    Returns (agg or None, dx2, agg_overflow, max_abs_agg)."""
    payloads = [np.ascontiguousarray(p) for p in payloads]
    pd = PAYLOAD_I8 if payloads[0].dtype == np.int8 else PAYLOAD_I32
    count = payloads[0].shape[0]
    assert x.dtype == np.float32 and x.flags.c_contiguous
    agg = np.empty(count, dtype=np.int32) if want_agg else None
    dx2, ovf, mx = C.c_double(), C.c_uint64(0), C.c_int32(0)
    lib().orc_aggregate(_ptr_array(payloads), pd, len(payloads), count, float(c), _ptr(x),
                        _ptr(agg), C.byref(dx2), C.byref(ovf), C.byref(mx))
    return agg, dx2.value, ovf.value, mx.value


def exact_step(grads, x, eta):
    """Init line of Algorithm 1: x <- x - eta * mean_i g_i.  Returns dx2."""
    grads = [np.ascontiguousarray(g) for g in grads]
    dx2 = C.c_double()
    lib().orc_exact_step(_ptr_array(grads), _grad_dtype(grads[0]), len(grads), x.shape[0],
                         float(eta), _ptr(x), C.byref(dx2))
    return dx2.value


def sqdiff(x, x_prev) -> float:
    x = np.ascontiguousarray(x, dtype=np.float32)
    x_prev = np.ascontiguousarray(x_prev, dtype=np.float32)
    return float(lib().orc_sqdiff(_ptr(x), _ptr(x_prev), x.shape[0]))


def step_window(grads, x, alpha, c, *, step, seed, j0=0, clip_limit=None,
                payload_dtype=PAYLOAD_I32, rounding=ROUND_RANDOM, want_agg=True):
    """One compressed step on coordinates [j0, j0 + len(x)) with (alpha, c) given.

    ``grads[i]`` and ``x`` hold only the window.  Updates x in place and returns a dict with
    agg, dx2 (of the window), clip_count[n], nonfinite, agg_overflow, max_abs_agg."""
    grads = [np.ascontiguousarray(g) for g in grads]
    n, count = len(grads), x.shape[0]
    if clip_limit is None:
        clip_limit = default_clip_limit(n, payload_dtype)
    agg = np.empty(count, dtype=np.int32) if want_agg else None
    scratch = np.empty(n * count, dtype=np.int32)
    clip = (C.c_uint64 * n)()
    dx2, nonf, ovf, mx = C.c_double(), C.c_uint64(0), C.c_uint64(0), C.c_int32(0)
    lib().orc_step_window(_ptr_array(grads), _grad_dtype(grads[0]), n, j0, count, float(alpha),
                          float(c), int(clip_limit), payload_dtype, rounding, seed, step, _ptr(x),
                          _ptr(agg), _ptr(scratch), C.byref(dx2), clip, C.byref(nonf),
                          C.byref(ovf), C.byref(mx))
    return dict(agg=agg, dx2=dx2.value, clip_count=[int(v) for v in clip], nonfinite=nonf.value,
                agg_overflow=ovf.value, max_abs_agg=mx.value)


class OracleIntSGD:
    """Algorithm 1 as a state machine: (r, dx2, step) carried between calls.

    ``step == 0`` is the exact first communication (Init line); every later step computes r_k and
    alpha_k (Proposition 2), rounds, sums, decodes and updates.  ``alpha_c`` lets a caller impose
    the fp32 (alpha, c) pair actually used for the vector part (lock-step comparison with an
    implementation whose norm reduction has another summation order); the oracle's own r and
    alpha are still computed and returned.
    """

    def __init__(self, n, d, *, beta=0.9, eps=1e-8, seed=0, payload_dtype=PAYLOAD_I32,
                 clip_limit=None, rounding=ROUND_RANDOM):
        self.n, self.d = n, d
        self.beta, self.eps, self.seed = beta, eps, seed
        self.payload_dtype, self.rounding = payload_dtype, rounding
        self.clip_limit = default_clip_limit(n, payload_dtype) if not clip_limit else clip_limit
        self.r = 0.0
        self.dx2 = 0.0
        self.step = 0

    def exact_step(self, grads, x, eta):
        dx2 = exact_step(grads, x, eta)
        self.dx2 = dx2
        self.step += 1
        return dict(dx2=dx2)

    def scale(self, eta, dx2=None):
        """Advance r with the stored (or given) squared step length and return the scale."""
        r, a64, a32, c32 = scale(self.d, self.n, eta, self.beta, self.eps, self.r,
                                 self.dx2 if dx2 is None else dx2)
        self.r = r
        return r, a64, a32, c32

    def int_step(self, grads, x, eta, *, alpha_c=None, dx2_in=None, want_agg=True):
        r, a64, a32, c32 = self.scale(eta, dx2_in)
        alpha, c = (a32, c32) if alpha_c is None else alpha_c
        out = step_window(grads, x, alpha, c, step=self.step, seed=self.seed, j0=0,
                          clip_limit=self.clip_limit, payload_dtype=self.payload_dtype,
                          rounding=self.rounding, want_agg=want_agg)
        self.dx2 = out["dx2"]
        self.step += 1
        out.update(r=r, alpha64=a64, alpha=a32, c=c32)
        return out


class OracleIntSGDBlocks:
    """Algorithm 2 (adaptive block quantization): one moving average r_{k,l} and one scale
    alpha_{k,l} = eta sqrt(d_l) / sqrt(2 n r_{k,l} + eta^2 (d_l / d) eps^2) per block l of
    coordinates [offsets[l], offsets[l+1]).  Each block is rounded, summed, decoded and applied with
    its own scale; the random stream is still indexed by the absolute coordinate.  Step 0 is the
    exact first communication, as in Algorithm 1.
    """

    def __init__(self, n, offsets, *, beta=0.9, eps=1e-8, seed=0, payload_dtype=PAYLOAD_I32,
                 clip_limit=None, rounding=ROUND_RANDOM):
        self.offsets = [int(o) for o in offsets]
        assert self.offsets[0] == 0 and all(a < b for a, b in zip(self.offsets, self.offsets[1:]))
        self.n, self.d, self.B = n, self.offsets[-1], len(self.offsets) - 1
        self.beta, self.eps, self.seed = beta, eps, seed
        self.payload_dtype, self.rounding = payload_dtype, rounding
        self.clip_limit = default_clip_limit(n, payload_dtype) if not clip_limit else clip_limit
        self.r = [0.0] * self.B
        self.dx2 = [0.0] * self.B
        self.step = 0

    def _block_dx2(self, x_new, x_old):
        return [sqdiff(x_new[a:b], x_old[a:b]) for a, b in zip(self.offsets, self.offsets[1:])]

    def exact_step(self, grads, x, eta):
        x_old = x.copy()
        exact_step(grads, x, eta)
        self.dx2 = self._block_dx2(x, x_old)
        self.step += 1
        return dict(dx2=list(self.dx2))

    def scales(self, eta, dx2=None):
        dx2 = self.dx2 if dx2 is None else dx2
        out = []
        for l, (a, b) in enumerate(zip(self.offsets, self.offsets[1:])):
            out.append(scale_block(self.d, b - a, self.n, eta, self.beta, self.eps, self.r[l], dx2[l]))
        return out   # list of (r, alpha64, alpha32, c32)

    def int_step(self, grads, x, eta, *, alpha_c=None, want_agg=True):
        """alpha_c: optional list of (alpha32, c32) per block imposed on the vector part."""
        sc = self.scales(eta)
        self.r = [t[0] for t in sc]
        agg = np.empty(self.d, dtype=np.int32) if want_agg else None
        clip = [0] * self.n
        nonf = ovf = mx = 0
        new_dx2 = []
        for l, (a, b) in enumerate(zip(self.offsets, self.offsets[1:])):
            alpha, c = (sc[l][2], sc[l][3]) if alpha_c is None else alpha_c[l]
            xw = x[a:b]   # a view: updated in place
            out = step_window([g[a:b] for g in grads], xw, alpha, c, step=self.step, seed=self.seed, j0=a,
                              clip_limit=self.clip_limit, payload_dtype=self.payload_dtype,
                              rounding=self.rounding, want_agg=want_agg)
            if want_agg:
                agg[a:b] = out["agg"]
            clip = [u + v for u, v in zip(clip, out["clip_count"])]
            nonf += out["nonfinite"]
            ovf += out["agg_overflow"]
            mx = max(mx, out["max_abs_agg"])
            new_dx2.append(out["dx2"])
        self.dx2 = new_dx2
        self.step += 1
        return dict(agg=agg, dx2=list(new_dx2), r=list(self.r), alpha64=[t[1] for t in sc],
                    alpha=[t[2] for t in sc], c=[t[3] for t in sc], clip_count=clip, nonfinite=nonf,
                    agg_overflow=ovf, max_abs_agg=mx)


def diana_factors(n, alpha, eta):
    """fp32 factors of an IntDIANA step for a given fp32 alpha: 1/alpha, 1/(n alpha), eta."""
    a = float(np.float32(alpha))
    return np.float32(1.0 / a), np.float32(1.0 / (float(n) * a)), np.float32(eta)


def diana_step_window(grads, h_local, h_global, x, alpha, eta, *, step, seed, j0=0, clip_limit=None,
                      payload_dtype=PAYLOAD_I32, rounding=ROUND_RANDOM, want_agg=True):
    """One IntDIANA step (Algorithm 3) on coordinates [j0, j0 + len(x)) with alpha given.

    Updates h_local[i], h_global and x in place; returns agg, dx2 and the counters."""
    grads = [np.ascontiguousarray(g) for g in grads]
    n, count = len(grads), x.shape[0]
    if clip_limit is None:
        clip_limit = default_clip_limit(n, payload_dtype)
    ainv, cn, eta32 = diana_factors(n, alpha, eta)
    agg = np.empty(count, dtype=np.int32) if want_agg else None
    clip = (C.c_uint64 * n)()
    dx2, nonf, ovf, mx = C.c_double(), C.c_uint64(0), C.c_uint64(0), C.c_int32(0)
    for h in list(h_local) + [h_global, x]:
        assert h.dtype == np.float32 and h.flags.c_contiguous and h.shape[0] == count
    lib().orc_diana_step_window(_ptr_array(grads), _grad_dtype(grads[0]), n, j0, count, float(np.float32(alpha)),
                                float(ainv), float(cn), float(eta32), int(clip_limit), payload_dtype, rounding,
                                seed, step, _ptr_array(h_local), _ptr(h_global), _ptr(x), _ptr(agg),
                                C.byref(dx2), clip, C.byref(nonf), C.byref(ovf), C.byref(mx))
    return dict(agg=agg, dx2=dx2.value, clip_count=[int(v) for v in clip], nonfinite=nonf.value,
                agg_overflow=ovf.value, max_abs_agg=mx.value)


class OracleIntDIANA:
    """Algorithm 3 as a state machine.  Step 0 is the exact mean step with h_i = h = 0; later steps
    use the scale rule of the context (Algorithm 3 prints its beta = 0, eps = 0 case,
    alpha_k = eta sqrt(d) / (sqrt(2n) ||x^k - x^{k-1}||))."""

    def __init__(self, n, d, *, beta=0.0, eps=0.0, seed=0, payload_dtype=PAYLOAD_I32, clip_limit=None,
                 rounding=ROUND_RANDOM):
        self.n, self.d, self.beta, self.eps, self.seed = n, d, beta, eps, seed
        self.payload_dtype, self.rounding = payload_dtype, rounding
        self.clip_limit = default_clip_limit(n, payload_dtype) if not clip_limit else clip_limit
        self.h_local = [np.zeros(d, dtype=np.float32) for _ in range(n)]
        self.h_global = np.zeros(d, dtype=np.float32)
        self.r, self.dx2, self.step = 0.0, 0.0, 0

    def exact_step(self, grads, x, eta):
        self.dx2 = exact_step(grads, x, eta)
        self.step += 1
        return dict(dx2=self.dx2)

    def int_step(self, grads, x, eta, *, alpha=None, want_agg=True):
        r, a64, a32, c32 = scale(self.d, self.n, eta, self.beta, self.eps, self.r, self.dx2)
        self.r = r
        out = diana_step_window(grads, self.h_local, self.h_global, x, a32 if alpha is None else alpha, eta,
                                step=self.step, seed=self.seed, clip_limit=self.clip_limit,
                                payload_dtype=self.payload_dtype, rounding=self.rounding, want_agg=want_agg)
        self.dx2 = out["dx2"]
        self.step += 1
        out.update(r=r, alpha64=a64, alpha=a32)
        return out


def heuristic_scale(grads, n, nb, eta):
    """Heuristic IntSGD scale (Section 5.2): profiling pass for the largest |g| over all workers (NaN
    ignored), then alpha = (2^nb - 1) / (n 2^max_exp).  Returns (max_abs, max_exp, alpha32, c32) or
    None when no scale exists (all zero, or an infinite entry)."""
    biggest = np.float32(0.0)
    for g in grads:
        g = np.ascontiguousarray(g)
        g32 = (g.astype(np.uint32) << 16).view(np.float32) if g.dtype == np.uint16 else g
        m = np.fmax.reduce(np.abs(g32), initial=np.float32(0.0))     # fmax ignores NaN
        biggest = np.fmax(biggest, m)
    e, a, c = C.c_int32(), C.c_float(), C.c_float()
    rc = lib().orc_heuristic_scale(float(biggest), n, nb, float(eta), C.byref(e), C.byref(a), C.byref(c))
    if rc != 0:
        return None
    return float(biggest), e.value, np.float32(a.value), np.float32(c.value)
