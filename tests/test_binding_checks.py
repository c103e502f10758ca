"""Host-side argument checks of the Python binding: a harness mistake (a short list, a wrong element type,
a host tensor, a short or strided buffer) must become an exception before any address reaches the C ABI.
No GPU is needed: the checks run before the library is called, so the context here is a stand-in object
whose C handle is never used."""
import numpy as np
import pytest
import torch

import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import binding


class _NeverCalled:
    def __getattr__(self, name):
        raise AssertionError(f"the C library was reached ({name}) although an argument was invalid")


def make(n=2, d=64, grad_dtype=pkg.GRAD_F32, payload_dtype=pkg.PAYLOAD_I32, device=0):
    obj = binding.IntSGD.__new__(binding.IntSGD)
    obj._lib, obj._ctx = _NeverCalled(), None
    obj.n, obj.d, obj.num_blocks = n, d, 0
    obj._g = "bf16" if grad_dtype == pkg.GRAD_BF16 else "f32"
    obj._p = "i8" if payload_dtype == pkg.PAYLOAD_I8 else "i32"
    obj._dev = device
    return obj


class FakeCuda:
    """Looks like a contiguous CUDA tensor to the checks; has no memory behind it."""
    def __init__(self, numel, dtype, index=0, contiguous=True):
        self._n, self.dtype, self.is_cuda, self._c = numel, dtype, True, contiguous
        self.device = torch.device("cuda", index)

    def numel(self):
        return self._n

    def is_contiguous(self):
        return self._c

    def data_ptr(self):
        raise AssertionError("the address of an invalid argument was taken")


def expect_invalid(fn, needle):
    with pytest.raises(pkg.IntSGDError) as e:
        fn()
    assert e.value.code == pkg.ERR_INVALID_ARG and needle in str(e.value), str(e.value)


def test_a_short_list_is_refused():
    lib, d = make(n=3), 64
    g = [FakeCuda(d, torch.float32) for _ in range(2)]
    x = FakeCuda(d, torch.float32)
    expect_invalid(lambda: lib.intsgd_step(g, x, None, eta_k=0.1), "n = 3")
    expect_invalid(lambda: lib.intsgd_aggregate([FakeCuda(d, torch.int32)], x), "n = 3")
    expect_invalid(lambda: lib.intsgd_diana_step(g + g, g + g[:1], x, x, eta_k=0.1), "n = 3")
    expect_invalid(lambda: lib.intsgd_step(g + g[:1], x, None, eta_k=0.1, mode=pkg.MODE_TWO_KERNEL,
                                           payload_scratch=[FakeCuda(d, torch.int32)]), "payload_scratch")


def test_a_wrong_element_type_is_refused():
    lib, d = make(n=1), 64
    x = FakeCuda(d, torch.float32)
    expect_invalid(lambda: lib.intsgd_step([FakeCuda(d, torch.float64)], x, None, eta_k=0.1), "float64")
    expect_invalid(lambda: lib.intsgd_step([FakeCuda(d, torch.bfloat16)], x, None, eta_k=0.1), "bfloat16")
    expect_invalid(lambda: lib.intsgd_step([x], FakeCuda(d, torch.float16), None, eta_k=0.1), "x:")
    expect_invalid(lambda: lib.intsgd_step([x], x, FakeCuda(d, torch.int64), eta_k=0.1), "agg")
    expect_invalid(lambda: lib.intsgd_encode(0, x, FakeCuda(d, torch.int8)), "payload")
    lib8 = make(n=1, grad_dtype=pkg.GRAD_BF16, payload_dtype=pkg.PAYLOAD_I8)
    expect_invalid(lambda: lib8.intsgd_encode(0, x, FakeCuda(d, torch.int8)), "grad")
    expect_invalid(lambda: lib8.intsgd_encode(0, FakeCuda(d, torch.bfloat16), FakeCuda(d, torch.int32)), "payload")


def test_host_tensors_short_buffers_and_other_devices_are_refused():
    lib, d = make(n=1), 64
    x = FakeCuda(d, torch.float32)
    expect_invalid(lambda: lib.intsgd_step([torch.zeros(d)], x, None, eta_k=0.1), "host buffer")
    expect_invalid(lambda: lib.intsgd_step([np.zeros(d, dtype=np.float32)], x, None, eta_k=0.1), "host buffer")
    expect_invalid(lambda: lib.intsgd_step([FakeCuda(d - 1, torch.float32)], x, None, eta_k=0.1), "63 elements")
    expect_invalid(lambda: lib.intsgd_step([x], FakeCuda(d, torch.float32, index=1), None, eta_k=0.1), "cuda:1")
    expect_invalid(lambda: lib.intsgd_step([FakeCuda(d, torch.float32, contiguous=False)], x, None, eta_k=0.1), "contiguous")
    expect_invalid(lambda: lib.intsgd_sqdiff(x, torch.zeros(d)), "x_prev")
    expect_invalid(lambda: lib.intsgd_heuristic_step([x], x, FakeCuda(3, torch.int32), eta_k=0.1, num_bits=8), "agg")


def test_step_host_wants_host_buffers():
    lib, d = make(n=1), 64
    hx = torch.zeros(d)
    expect_invalid(lambda: lib.intsgd_step_host([FakeCuda(d, torch.float32)], hx, None, eta_k=0.1), "device tensor")
    expect_invalid(lambda: lib.intsgd_step_host([torch.zeros(d)], torch.zeros(d - 1), None, eta_k=0.1), "host_x")
    expect_invalid(lambda: lib.intsgd_step_host([torch.zeros(d)], hx, torch.zeros(d, dtype=torch.int16), eta_k=0.1), "host_agg")
    expect_invalid(lambda: lib.intsgd_step_host([torch.zeros(d)[::2]], hx, None, eta_k=0.1), "host_grads[0]")
    expect_invalid(lambda: lib.intsgd_step_host([], hx, None, eta_k=0.1), "n = 1")


def test_sqdiff_noalloc_checks_length_and_output_type(monkeypatch):
    monkeypatch.setattr(binding, "load", lambda: _NeverCalled())
    d = 32
    x = FakeCuda(d, torch.float32)
    expect_invalid(lambda: pkg.intsgd_sqdiff_noalloc(x, x, d + 1, FakeCuda(1, torch.float64)), "33")
    expect_invalid(lambda: pkg.intsgd_sqdiff_noalloc(x, x, d, FakeCuda(1, torch.float32)), "out")
    expect_invalid(lambda: pkg.intsgd_sqdiff_noalloc(x, torch.zeros(d), d, FakeCuda(1, torch.float64)), "x_prev")
    expect_invalid(lambda: pkg.intsgd_sqdiff_noalloc(FakeCuda(d, torch.float64), x, d, FakeCuda(1, torch.float64)), "float64")
