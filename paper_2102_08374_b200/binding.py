"""Thin ctypes binding of ``libintsgd.so`` (the C ABI declared in ``include/intsgd.h``).

Argument marshalling only: every step of the IntSGD path runs in the CUDA kernels.  Before an address
crosses the C ABI the binding checks what the library cannot see from a bare pointer: the number of
buffers in a list, element type, length, contiguity and which device a tensor lives on
(``IntSGDError`` with ``ERR_INVALID_ARG``; nothing is launched).  There is no
CPU fallback; if the library cannot be loaded, or no CUDA device is present when a context is
created, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import math
from pathlib import Path

from . import buildlib as _build

MAX_WORKERS = 64

OK = 0
ERR_INVALID_ARG = -1
ERR_ALIGN = -2
ERR_CUDA = -3
ERR_SCALE_NONFINITE = -4
ERR_UNSUPPORTED = -5
ERR_TIMEOUT = -6
ERR_TOO_LARGE = -7
NOALLOC_MAX_D = 1 << 28

GRAD_F32, GRAD_BF16 = 0, 1
PAYLOAD_I32, PAYLOAD_I8 = 0, 1
ROUND_RANDOM, ROUND_NEAREST, ROUND_RANDOM16, ROUND_RANDOM_COMPARE = 0, 1, 2, 3
MODE_EXACT, MODE_TWO_KERNEL, MODE_FUSED = 0, 1, 2

EXPORTS = [
    "intsgd_create", "intsgd_destroy", "intsgd_scale", "intsgd_sqdiff", "intsgd_encode",
    "intsgd_aggregate", "intsgd_step", "intsgd_step_host", "intsgd_get_stats", "intsgd_get_state",
    "intsgd_set_state", "intsgd_set_launch", "intsgd_set_fused_path", "intsgd_launch_count", "intsgd_last_error",
    "intsgd_sqdiff_noalloc", "intsgd_set_blocks", "intsgd_get_block_state", "intsgd_set_block_state",
    "intsgd_diana_step", "intsgd_heuristic_step", "intsgd_selftest_wait_expiry", "intsgd_selftest_philox_rate",
]


class Config(C.Structure):
    _fields_ = [("n", C.c_int32), ("grad_dtype", C.c_int32), ("d", C.c_int64),
                ("payload_dtype", C.c_int32), ("rounding", C.c_int32), ("beta", C.c_double),
                ("eps", C.c_double), ("seed", C.c_uint64), ("clip_limit", C.c_int64),
                ("device", C.c_int32), ("reserved", C.c_int32)]


class State(C.Structure):
    _fields_ = [("r", C.c_double), ("dx2", C.c_double), ("alpha", C.c_float), ("c", C.c_float),
                ("step", C.c_uint32), ("status", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("state", State), ("clip_count", C.c_uint64 * MAX_WORKERS), ("nonfinite", C.c_uint64),
                ("agg_overflow", C.c_uint64), ("max_abs_agg", C.c_int32), ("reserved", C.c_int32)]


class IntSGDError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"intsgd error {code}: {message}")
        self.code = code


_lib = None


def library_path() -> Path:
    return _build.LIB


def load() -> C.CDLL:
    """Load ``libintsgd.so`` (building it with nvcc first if it is absent)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not path.exists():
        _build.build()
    lib = C.CDLL(str(path))
    vp, i32, i64, f64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_double, C.c_float
    lib.intsgd_create.argtypes = [C.POINTER(vp), C.POINTER(Config)]
    lib.intsgd_destroy.argtypes = [vp]
    lib.intsgd_scale.argtypes = [vp, f64, f64, vp]
    lib.intsgd_sqdiff.argtypes = [vp, vp, vp, vp]
    lib.intsgd_encode.argtypes = [vp, i32, vp, vp, f32, vp]
    lib.intsgd_aggregate.argtypes = [vp, C.POINTER(vp), vp, vp, vp]
    lib.intsgd_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, vp, f64, i32, vp]
    lib.intsgd_diana_step.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), vp, vp, vp, f64, vp]
    lib.intsgd_heuristic_step.argtypes = [vp, C.POINTER(vp), vp, vp, f64, i32, vp]
    lib.intsgd_step_host.argtypes = [vp, C.POINTER(vp), vp, vp, f64, i32, vp]
    lib.intsgd_get_stats.argtypes = [vp, C.POINTER(Stats)]
    lib.intsgd_get_state.argtypes = [vp, C.POINTER(State)]
    lib.intsgd_set_state.argtypes = [vp, C.POINTER(State)]
    lib.intsgd_set_launch.argtypes = [vp, i32, i32]
    lib.intsgd_set_fused_path.argtypes = [vp, i32]
    lib.intsgd_set_blocks.argtypes = [vp, i32, C.POINTER(C.c_int64)]
    lib.intsgd_get_block_state.argtypes = [vp, vp, vp, vp, vp]
    lib.intsgd_set_block_state.argtypes = [vp, vp, vp]
    lib.intsgd_sqdiff_noalloc.argtypes = [vp, vp, i64, vp, vp]
    lib.intsgd_selftest_wait_expiry.argtypes = [vp, vp]
    lib.intsgd_selftest_philox_rate.argtypes = [vp, i64, i32, C.POINTER(i64), vp]
    lib.intsgd_launch_count.argtypes = [vp]
    lib.intsgd_launch_count.restype = i64
    lib.intsgd_last_error.argtypes = [vp]
    lib.intsgd_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("intsgd_launch_count", "intsgd_last_error"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _addr(t) -> int | None:
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    if hasattr(t, "ctypes"):
        return t.ctypes.data
    raise TypeError(f"cannot take the address of {type(t)}")


# Element types a buffer may have for each role.  bf16 gradients may also be handed over as their 16-bit
# patterns (int16 / uint16 carriers).
_DTYPES = {
    "f32": ("float32",), "bf16": ("bfloat16", "int16", "uint16"), "i32": ("int32",), "i8": ("int8",),
    "f64": ("float64",),
}


def _bad(msg: str):
    raise IntSGDError(ERR_INVALID_ARG, msg)


def _check_buffer(t, what: str, kind: str, count: int, device: int | None):
    """Host-side argument check of one vector before its address crosses the C ABI.

    ``device`` is the CUDA ordinal the buffer must live on, or None for a host buffer.  A raw integer
    address cannot be inspected and is passed through (the library still checks NULL and alignment);
    None is left to the library as well, which reports it as a NULL pointer.
    """
    if t is None or isinstance(t, int):
        return
    name = str(getattr(t, "dtype", "")).replace("torch.", "")
    if name not in _DTYPES[kind]:
        _bad(f"{what}: element type {name or type(t).__name__} where {' / '.join(_DTYPES[kind])} is expected")
    numel = t.numel() if hasattr(t, "numel") else int(getattr(t, "size", 0))
    if numel < count:
        _bad(f"{what}: {numel} elements where at least {count} are needed")
    if hasattr(t, "is_contiguous"):
        if not t.is_contiguous():
            _bad(f"{what}: not contiguous")
    elif hasattr(t, "flags") and not t.flags["C_CONTIGUOUS"]:
        _bad(f"{what}: not contiguous")
    on_cuda = bool(getattr(t, "is_cuda", False))
    if device is None:
        if on_cuda:
            _bad(f"{what}: a device tensor where a host buffer is expected")
    else:
        if not on_cuda:
            _bad(f"{what}: a host buffer where a tensor on cuda:{device} is expected")
        if t.device.index != device:
            _bad(f"{what}: lives on cuda:{t.device.index}, the context is on cuda:{device}")


def _check_list(seq, what: str, kind: str, count: int, device: int | None, n: int):
    if seq is None or len(seq) != n:
        _bad(f"{what}: {0 if seq is None else len(seq)} buffers where the context has n = {n} workers")
    for i, t in enumerate(seq):
        _check_buffer(t, f"{what}[{i}]", kind, count, device)


def _ptr_array(seq):
    return (C.c_void_p * len(seq))(*[_addr(t) for t in seq])


def intsgd_sqdiff_noalloc(x, x_prev, d, out, stream=None) -> None:
    """``out[0] = ||x - x_prev||^2`` on the current device without any device allocation.

    For hosts that cannot create a context (``intsgd_create`` calls ``cudaMalloc``): the reduction
    scratch is a fixed 128 KiB array inside the library.  ``x``, ``x_prev``: d floats on the device;
    ``out``: one device double.  ``d`` may not exceed ``NOALLOC_MAX_D``.  Calls on one device share
    the scratch, so they must not overlap on the GPU.
    """
    if isinstance(d, int) and 1 <= d <= NOALLOC_MAX_D:   # other sizes are refused by the library itself
        where = next((t.device.index for t in (x, x_prev, out) if getattr(t, "is_cuda", False)), 0)
        _check_buffer(x, "x", "f32", d, where)
        _check_buffer(x_prev, "x_prev", "f32", d, where)
        _check_buffer(out, "out", "f64", 1, where)
    rc = load().intsgd_sqdiff_noalloc(_addr(x), _addr(x_prev), d, _addr(out), stream)
    if rc != OK:
        what = {ERR_TOO_LARGE: f"d = {d} exceeds the fixed scratch (max {NOALLOC_MAX_D} coordinates)",
                ERR_INVALID_ARG: "null pointer or d < 1", ERR_ALIGN: "pointer not aligned to its element size",
                ERR_CUDA: "a CUDA runtime call failed"}.get(rc, "failed")
        raise IntSGDError(rc, f"intsgd_sqdiff_noalloc: {what}")


class IntSGD:
    """One IntSGD context.  Method names and arguments mirror the C ABI one to one."""

    def __init__(self, n, d, *, grad_dtype=GRAD_F32, payload_dtype=PAYLOAD_I32,
                 rounding=ROUND_RANDOM, beta=0.9, eps=1e-8, seed=0, clip_limit=0, device=0):
        self._lib = load()
        self.cfg = Config(n=n, grad_dtype=grad_dtype, d=d, payload_dtype=payload_dtype,
                          rounding=rounding, beta=beta, eps=eps, seed=seed, clip_limit=clip_limit,
                          device=device, reserved=0)
        self._ctx = C.c_void_p()
        rc = self._lib.intsgd_create(C.byref(self._ctx), C.byref(self.cfg))
        if rc != OK:
            msg = self._lib.intsgd_last_error(None).decode()
            self._ctx = C.c_void_p()
            raise IntSGDError(rc, msg)
        self.n, self.d = n, d
        self.num_blocks = 0
        self._g = "bf16" if grad_dtype == GRAD_BF16 else "f32"
        self._p = "i8" if payload_dtype == PAYLOAD_I8 else "i32"
        self._dev = device

    # -- lifetime ---------------------------------------------------------------------------
    def close(self):
        if getattr(self, "_ctx", None):
            self._lib.intsgd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _check(self, rc, allow=()):
        if rc != OK and rc not in allow:
            raise IntSGDError(rc, self._lib.intsgd_last_error(self._ctx).decode())
        return rc

    def _check_x_agg(self, x, agg):
        _check_buffer(x, "x", "f32", self.d, self._dev)
        _check_buffer(agg, "agg", "i32", self.d, self._dev)

    # -- the calls of the C ABI -----------------------------------------------------------------
    def intsgd_scale(self, eta_k, dx2_override=-1.0, stream=None):
        self._check(self._lib.intsgd_scale(self._ctx, eta_k, dx2_override, stream))

    def intsgd_sqdiff(self, x, x_prev, stream=None):
        _check_buffer(x, "x", "f32", self.d, self._dev)
        _check_buffer(x_prev, "x_prev", "f32", self.d, self._dev)
        self._check(self._lib.intsgd_sqdiff(self._ctx, _addr(x), _addr(x_prev), stream))

    def intsgd_encode(self, worker, grad, payload, alpha_override=math.nan, stream=None):
        _check_buffer(grad, "grad", self._g, self.d, self._dev)
        _check_buffer(payload, "payload", self._p, self.d, self._dev)
        self._check(self._lib.intsgd_encode(self._ctx, worker, _addr(grad), _addr(payload),
                                            alpha_override, stream))

    def intsgd_aggregate(self, payloads, x, agg=None, stream=None):
        _check_list(payloads, "payloads", self._p, self.d, self._dev, self.n)
        self._check_x_agg(x, agg)
        self._check(self._lib.intsgd_aggregate(self._ctx, _ptr_array(payloads), _addr(x), _addr(agg), stream))

    def intsgd_step(self, grads, x, agg=None, *, eta_k, mode=MODE_FUSED, payload_scratch=None, stream=None):
        _check_list(grads, "grads", self._g, self.d, self._dev, self.n)
        self._check_x_agg(x, agg)
        if payload_scratch is not None:
            _check_list(payload_scratch, "payload_scratch", self._p, self.d, self._dev, self.n)
        scratch = _ptr_array(payload_scratch) if payload_scratch is not None else None
        self._check(self._lib.intsgd_step(self._ctx, _ptr_array(grads), scratch, _addr(x), _addr(agg),
                                          eta_k, mode, stream))

    def intsgd_diana_step(self, grads, h_local, h_global, x, agg=None, *, eta_k, stream=None):
        _check_list(grads, "grads", self._g, self.d, self._dev, self.n)
        _check_list(h_local, "h_local", "f32", self.d, self._dev, self.n)
        _check_buffer(h_global, "h_global", "f32", self.d, self._dev)
        self._check_x_agg(x, agg)
        self._check(self._lib.intsgd_diana_step(self._ctx, _ptr_array(grads), _ptr_array(h_local), _addr(h_global),
                                                _addr(x), _addr(agg), eta_k, stream))

    def intsgd_heuristic_step(self, grads, x, agg=None, *, eta_k, num_bits, stream=None):
        _check_list(grads, "grads", self._g, self.d, self._dev, self.n)
        self._check_x_agg(x, agg)
        self._check(self._lib.intsgd_heuristic_step(self._ctx, _ptr_array(grads), _addr(x), _addr(agg), eta_k,
                                                    num_bits, stream))

    def intsgd_step_host(self, host_grads, host_x, host_agg=None, *, eta_k, mode=MODE_FUSED, stream=None):
        _check_list(host_grads, "host_grads", self._g, self.d, None, self.n)
        _check_buffer(host_x, "host_x", "f32", self.d, None)
        _check_buffer(host_agg, "host_agg", "i32", self.d, None)
        self._check(self._lib.intsgd_step_host(self._ctx, _ptr_array(host_grads), _addr(host_x),
                                               _addr(host_agg), eta_k, mode, stream))

    def intsgd_get_stats(self, allow_nonfinite=False) -> dict:
        s = Stats()
        rc = self._check(self._lib.intsgd_get_stats(self._ctx, C.byref(s)),
                         allow=(ERR_SCALE_NONFINITE,) if allow_nonfinite else ())
        st = s.state
        return dict(rc=rc, r=st.r, dx2=st.dx2, alpha=st.alpha, c=st.c, step=st.step, status=st.status,
                    clip_count=[int(v) for v in s.clip_count[: self.n]], nonfinite=int(s.nonfinite),
                    agg_overflow=int(s.agg_overflow), max_abs_agg=int(s.max_abs_agg))

    def intsgd_get_state(self) -> State:
        st = State()
        self._check(self._lib.intsgd_get_state(self._ctx, C.byref(st)), allow=(ERR_SCALE_NONFINITE,))
        return st

    def intsgd_set_state(self, *, r, dx2, alpha, c, step, status=OK):
        st = State(r=r, dx2=dx2, alpha=alpha, c=c, step=step, status=status)
        self._check(self._lib.intsgd_set_state(self._ctx, C.byref(st)))

    def intsgd_set_launch(self, threads_per_block=0, blocks_per_sm=0):
        self._check(self._lib.intsgd_set_launch(self._ctx, threads_per_block, blocks_per_sm))

    def intsgd_set_blocks(self, offsets):
        """Block partition for Algorithm 2; ``offsets`` has num_blocks + 1 entries (empty/None = off)."""
        offsets = list(offsets) if offsets is not None else []
        B = max(len(offsets) - 1, 0)
        arr = (C.c_int64 * (B + 1))(*offsets) if B else None
        self._check(self._lib.intsgd_set_blocks(self._ctx, B, arr))
        self.num_blocks = B

    def intsgd_get_block_state(self) -> dict:
        B = self.num_blocks
        r, dx2 = (C.c_double * B)(), (C.c_double * B)()
        alpha, c = (C.c_float * B)(), (C.c_float * B)()
        self._check(self._lib.intsgd_get_block_state(self._ctx, C.addressof(r), C.addressof(dx2),
                                                     C.addressof(alpha), C.addressof(c)))
        return dict(r=list(r), dx2=list(dx2), alpha=list(alpha), c=list(c))

    def intsgd_set_block_state(self, r=None, dx2=None):
        B = self.num_blocks
        ra = (C.c_double * B)(*r) if r is not None else None
        da = (C.c_double * B)(*dx2) if dx2 is not None else None
        self._check(self._lib.intsgd_set_block_state(self._ctx, C.addressof(ra) if ra is not None else None,
                                                     C.addressof(da) if da is not None else None))

    def intsgd_set_fused_path(self, path: int):
        self._check(self._lib.intsgd_set_fused_path(self._ctx, path))

    def intsgd_selftest_wait_expiry(self, stream=None):
        self._check(self._lib.intsgd_selftest_wait_expiry(self._ctx, stream))

    def intsgd_selftest_philox_rate(self, blocks_per_thread, extra_ops_per_block=0, stream=None) -> int:
        """Enqueue the register-only Philox kernel; returns the number of Philox blocks the launch computes."""
        count = C.c_int64(0)
        self._check(self._lib.intsgd_selftest_philox_rate(self._ctx, blocks_per_thread, extra_ops_per_block,
                                                          C.byref(count), stream))
        return int(count.value)

    def intsgd_launch_count(self) -> int:
        return int(self._lib.intsgd_launch_count(self._ctx))

    def intsgd_last_error(self) -> str:
        return self._lib.intsgd_last_error(self._ctx).decode()
