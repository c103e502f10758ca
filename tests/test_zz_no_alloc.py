"""intsgd_sqdiff_noalloc: the allocation-free norm entry point against intsgd_sqdiff and against the CPU oracle.

Collected last on purpose (file name): a failure here cannot hide a failure elsewhere.  The entry
point exists for hosts that cannot call cudaMalloc and therefore cannot create a context; its
scratch is a fixed array in the library that every call on the device shares, so the test calls it
twice in a row on different data and expects both answers to match the context-based entry point, and
the oracle's serial fp64 sum of the same vectors.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg

pytestmark = pytest.mark.gpu

REL = 1e-12   # the tolerance the intsgd_sqdiff tests use


def _reference(x, x_prev):
    d = x.numel()
    with pkg.IntSGD(1, d) as lib:
        lib.intsgd_sqdiff(x, x_prev)
        return lib.intsgd_get_stats()["dx2"]


def test_two_calls_in_a_row_match_the_context_entry_point():
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(123)
    out = torch.zeros(2, dtype=torch.float64, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    cases = [3 * (1 << 18) + 1, 16384 * 5 + 7]      # many blocks + ragged tail, then a shorter vector
    got, want = [], []
    pairs = []
    for d in cases:
        x = torch.randn(d, generator=gen, device=dev)
        x_prev = x + 1e-3 * torch.randn(d, generator=gen, device=dev)
        pairs.append((x, x_prev))
    # back to back on one stream: the second call starts from the first call's scratch contents
    for k, (x, x_prev) in enumerate(pairs):
        pkg.intsgd_sqdiff_noalloc(x, x_prev, x.numel(), out[k:], stream)
    torch.cuda.synchronize()
    got = out.cpu().tolist()
    want = [_reference(x, x_prev) for x, x_prev in pairs]
    for g, w in zip(got, want):
        assert w > 0 and abs(g - w) <= REL * w, (g, w)
    for g, (x, x_prev) in zip(got, pairs):   # and the oracle: serial fp64 sum of the squared fp32 differences
        w = oracle.sqdiff(x.cpu().numpy(), x_prev.cpu().numpy())
        assert abs(g - w) <= REL * w, (g, w)
    # an unaligned view (element-wise loads) and a repeat of the first case give the same answers
    x, x_prev = pairs[1]
    xb = torch.empty(x.numel() + 1, device=dev)[1:].copy_(x)
    pkg.intsgd_sqdiff_noalloc(xb, x_prev, x.numel(), out[:1], stream)
    pkg.intsgd_sqdiff_noalloc(pairs[0][0], pairs[0][1], pairs[0][0].numel(), out[1:], stream)
    torch.cuda.synchronize()
    again = out.cpu().tolist()
    assert abs(again[0] - want[1]) <= REL * want[1]
    assert again[1] == got[0]          # same d, same data: same summation order, same bits


def test_rejects_bad_sizes_and_pointers_without_touching_the_gpu():
    dev = torch.device("cuda:0")
    x = torch.zeros(8, device=dev)
    out = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
    with pytest.raises(pkg.IntSGDError) as e:
        pkg.intsgd_sqdiff_noalloc(x, x, pkg.NOALLOC_MAX_D + 1, out)
    assert e.value.code == pkg.ERR_TOO_LARGE and "exceeds" in str(e.value)
    for d in (0, -5):
        with pytest.raises(pkg.IntSGDError) as e:
            pkg.intsgd_sqdiff_noalloc(x, x, d, out)
        assert e.value.code == pkg.ERR_INVALID_ARG
    with pytest.raises(pkg.IntSGDError) as e:
        pkg.intsgd_sqdiff_noalloc(x, None, 8, out)
    assert e.value.code == pkg.ERR_INVALID_ARG
    with pytest.raises(pkg.IntSGDError) as e:
        pkg.intsgd_sqdiff_noalloc(x.data_ptr() + 2, x, 4, out)
    assert e.value.code == pkg.ERR_ALIGN
    torch.cuda.synchronize()
    assert out.item() == -1.0
