"""IntSGD step library for NVIDIA B200: CUDA kernels behind a C ABI, with a ctypes binding.

``IntSGD`` mirrors the entry points declared in ``include/intsgd.h``.  ``synth`` holds the
seeded synthetic workloads.  Importing this package loads nothing; the shared library is loaded
(and, if absent, built with nvcc) when the first context is created.
"""
from .binding import (  # noqa: F401
    ERR_ALIGN, ERR_CUDA, ERR_INVALID_ARG, ERR_SCALE_NONFINITE, ERR_TIMEOUT, ERR_TOO_LARGE, ERR_UNSUPPORTED, EXPORTS, GRAD_BF16,
    GRAD_F32, MAX_WORKERS, MODE_EXACT, MODE_FUSED, MODE_TWO_KERNEL, OK, PAYLOAD_I8, PAYLOAD_I32,
    NOALLOC_MAX_D, ROUND_NEAREST, ROUND_RANDOM, ROUND_RANDOM16, ROUND_RANDOM_COMPARE, IntSGD, IntSGDError, intsgd_sqdiff_noalloc, library_path, load,
)
from .buildlib import build  # noqa: F401
