"""Guard bands: every output buffer of the library sits inside a larger allocation filled with a sentinel,
and after each call the bytes before and after it must be untouched.  Algorithm 1's vectors have length
d and nothing may be written beyond them; the kernels' hand-written tails (the last < 8 coordinates of the
pipelined kernel, the "even units" rule of bf16 tiles, byte-packed int8 stores, 16-wide int8 loads, the
windows of the host-buffer step) are where an off-by-one would write one element too far and still
pass a parity test.  This is the stand-in for a memory checker."""
import numpy as np
import pytest
import torch

import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

pytestmark = pytest.mark.gpu

PAD = 512          # bytes on each side, a multiple of 16
SENTINEL = 0xA5


class Guarded:
    """A typed view of `numel` elements inside a sentinel-filled byte buffer.  shift = elements by which the
    view is moved off the 16-byte boundary (0 = 16-byte aligned)."""

    def __init__(self, numel, dtype, shift=0, device="cuda:0", pinned=False):
        self.item = torch.empty(0, dtype=dtype).element_size()
        nbytes = numel * self.item
        total = PAD + shift * self.item + nbytes + PAD + 16
        if device == "cpu":
            self.raw = torch.empty(total, dtype=torch.uint8, pin_memory=pinned)
        else:
            self.raw = torch.empty(total, dtype=torch.uint8, device=device)
        self.raw.fill_(SENTINEL)
        assert self.raw.data_ptr() % 16 == 0
        self.lo = PAD + shift * self.item
        self.hi = self.lo + nbytes
        self.t = self.raw[self.lo:self.hi].view(dtype)
        assert self.t.numel() == numel and (self.t.data_ptr() % 16 == 0) == (shift * self.item % 16 == 0)

    def check(self, what):
        before, after = self.raw[: self.lo].cpu().numpy(), self.raw[self.hi:].cpu().numpy()
        bad_b, bad_a = np.nonzero(before != SENTINEL)[0], np.nonzero(after != SENTINEL)[0]
        assert bad_b.size == 0, f"{what}: {bad_b.size} bytes written before the buffer (first at -{self.lo - int(bad_b[0])})"
        assert bad_a.size == 0, f"{what}: {bad_a.size} bytes written after the buffer (first at +{int(bad_a[0])})"

    def touched(self):
        """True if some byte of the payload is no longer the sentinel (the call did write its output)."""
        return bool((self.raw[self.lo:self.hi] != SENTINEL).any().item()) if self.hi > self.lo else True


def grads_for(n, d, bf16, seed=40):
    out = []
    for i in range(n):
        g = synth.bucket_gradient(i, d, seed_base=seed)
        if bf16:
            out.append(torch.from_numpy(synth.to_bf16_bits(g).view(np.int16)).cuda().view(torch.bfloat16))
        else:
            out.append(torch.from_numpy(g).cuda())
    return out


def fill(buf: Guarded, values: torch.Tensor):
    buf.t.copy_(values)


SIZES = [1, 3, 7, 12, 1023, (1 << 16) + 2, 8200 + 5, 2 * 1024 * 4 + 4 + 3]   # incl. odd unit counts for bf16


@pytest.mark.parametrize("d", SIZES)
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("shift", [0, 1])
@pytest.mark.parametrize("path", [0, 1])
def test_fused_and_exact_steps_stay_inside_x_and_agg(d, bf16, shift, path):
    n = 3
    g = grads_for(n, d, bf16)
    x = Guarded(d, torch.float32, shift)
    agg = Guarded(d, torch.int32, shift)
    fill(x, torch.from_numpy(synth.iterate(d, seed=41)).cuda())
    payload = pkg.PAYLOAD_I8 if (d % 2) else pkg.PAYLOAD_I32
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16 if bf16 else pkg.GRAD_F32, payload_dtype=payload, seed=5) as lib:
        lib.intsgd_set_fused_path(path)
        lib.intsgd_step(g, x.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        torch.cuda.synchronize()
        x.check("x after the exact step")
        agg.check("agg after the exact step (not an output of it)")
        assert not agg.touched()
        for k in range(2):
            lib.intsgd_step(g, x.t, agg.t, eta_k=0.1, mode=pkg.MODE_FUSED)
            lib.intsgd_get_stats()
            x.check(f"x after fused step {k}")
            agg.check(f"agg after fused step {k}")
        assert agg.touched()


@pytest.mark.parametrize("d", [1, 15, 17, 31, 1023, 4096 + 1, 4096 + 15, (1 << 16) + 2])
@pytest.mark.parametrize("pay", [pkg.PAYLOAD_I32, pkg.PAYLOAD_I8])
@pytest.mark.parametrize("shift", [0, 1, 3])
@pytest.mark.parametrize("bf16", [False, True])
def test_two_kernel_step_stays_inside_payloads_x_and_agg(d, pay, shift, bf16):
    n = 3
    g = grads_for(n, d, bf16, seed=50)
    x = Guarded(d, torch.float32, shift % 2)
    agg = Guarded(d, torch.int32, shift % 2)
    pt = torch.int8 if pay == pkg.PAYLOAD_I8 else torch.int32
    pays = [Guarded(d, pt, shift) for _ in range(n)]
    fill(x, torch.from_numpy(synth.iterate(d, seed=51)).cuda())
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16 if bf16 else pkg.GRAD_F32, payload_dtype=pay, seed=6) as lib:
        lib.intsgd_step(g, x.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        lib.intsgd_step(g, x.t, agg.t, eta_k=0.1, mode=pkg.MODE_TWO_KERNEL, payload_scratch=[p.t for p in pays])
        lib.intsgd_get_stats()
        for i, p in enumerate(pays):
            p.check(f"payload {i} after the two-kernel step")
            assert p.touched()
        x.check("x after the two-kernel step")
        agg.check("agg after the two-kernel step")
        # the separate calls: one worker's encode, then the aggregate
        lib.intsgd_scale(0.1)
        for i in range(n):
            lib.intsgd_encode(i, g[i], pays[i].t)
        lib.intsgd_aggregate([p.t for p in pays], x.t, agg.t)
        lib.intsgd_get_stats()
        for i, p in enumerate(pays):
            p.check(f"payload {i} after intsgd_encode")
        x.check("x after intsgd_aggregate")
        agg.check("agg after intsgd_aggregate")


@pytest.mark.parametrize("d", [1, 7, 1023, 8200 + 5, (1 << 16) + 2])
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("shift", [0, 1])
@pytest.mark.parametrize("path", [0, 1])
def test_diana_step_stays_inside_shifts_x_and_agg(d, bf16, shift, path):
    n = 3
    g = grads_for(n, d, bf16, seed=60)
    x, agg, h = Guarded(d, torch.float32, shift), Guarded(d, torch.int32, shift), Guarded(d, torch.float32, shift)
    hl = [Guarded(d, torch.float32, shift) for _ in range(n)]
    fill(x, torch.from_numpy(synth.iterate(d, seed=61)).cuda())
    h.t.zero_()
    for b in hl:
        b.t.zero_()
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16 if bf16 else pkg.GRAD_F32, seed=7) as lib:
        lib.intsgd_set_fused_path(path)
        lib.intsgd_step(g, x.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        for k in range(2):
            lib.intsgd_diana_step(g, [b.t for b in hl], h.t, x.t, agg.t, eta_k=0.1)
            lib.intsgd_get_stats()
            for i, b in enumerate(hl):
                b.check(f"local shift {i} after IntDIANA step {k}")
            h.check("global shift"); x.check("x"); agg.check("agg")


@pytest.mark.parametrize("d", [9, 1023, 8200 + 5, (1 << 16) + 2])
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("shift", [0, 1])
def test_block_wise_step_stays_inside_x_and_agg(d, bf16, shift):
    n = 3
    g = grads_for(n, d, bf16, seed=70)
    x, agg = Guarded(d, torch.float32, shift), Guarded(d, torch.int32, shift)
    fill(x, torch.from_numpy(synth.iterate(d, seed=71)).cuda())
    offsets = sorted({0, 1, d // 3, d // 3 + 5, (2 * d) // 3, d - 1, d})
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16 if bf16 else pkg.GRAD_F32, seed=8) as lib:
        lib.intsgd_set_blocks(offsets)
        lib.intsgd_step(g, x.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        for k in range(2):
            lib.intsgd_step(g, x.t, agg.t, eta_k=0.1, mode=pkg.MODE_FUSED)
            lib.intsgd_get_stats()
            x.check(f"x after block-wise step {k}")
            agg.check(f"agg after block-wise step {k}")


def test_heuristic_step_and_sqdiff_noalloc_stay_inside_their_outputs():
    n, d = 2, 8200 + 5
    g = grads_for(n, d, False, seed=80)
    x, agg = Guarded(d, torch.float32, 1), Guarded(d, torch.int32, 1)
    fill(x, torch.from_numpy(synth.iterate(d, seed=81)).cuda())
    with pkg.IntSGD(n, d, seed=9) as lib:
        lib.intsgd_step(g, x.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        for nb in (8, 31):
            lib.intsgd_heuristic_step(g, x.t, agg.t, eta_k=0.1, num_bits=nb)
            lib.intsgd_get_stats()
            x.check(f"x after the heuristic step ({nb} bits)")
            agg.check(f"agg after the heuristic step ({nb} bits)")
    out = Guarded(1, torch.float64)
    xp = torch.from_numpy(synth.iterate(d, seed=82)).cuda()
    for a, b in ((x.t, xp), (xp, xp + 1.0)):       # element-aligned and 16-byte aligned inputs
        pkg.intsgd_sqdiff_noalloc(a, b, d, out.t)
        torch.cuda.synchronize()
        out.check("out of intsgd_sqdiff_noalloc")
        assert out.t.item() > 0.0


@pytest.mark.parametrize("d,bf16", [(8 * (1 << 22) + 4101, False), ((1 << 22) + 4 + 2, True), (1023, False)])
def test_host_buffer_step_stays_inside_the_host_buffers(d, bf16):
    """The windowed host-buffer step (windows of 2^22 coordinates, a ragged last window) writes x and the
    aggregate back to host memory: the guard bands are around the HOST buffers."""
    n = 2
    rng = np.random.default_rng(90)
    hg = []
    for i in range(n):
        v = (rng.standard_normal(d, dtype=np.float32) * np.float32(1e-3))
        hg.append(torch.from_numpy(synth.to_bf16_bits(v).view(np.int16)) if bf16 else torch.from_numpy(v))
    hx = Guarded(d, torch.float32, 1, device="cpu")
    hagg = Guarded(d, torch.int32, 3, device="cpu")
    hx.t.copy_(torch.from_numpy(rng.standard_normal(d, dtype=np.float32)))
    with pkg.IntSGD(n, d, grad_dtype=pkg.GRAD_BF16 if bf16 else pkg.GRAD_F32, seed=10) as lib:
        lib.intsgd_step_host(hg, hx.t, None, eta_k=0.1, mode=pkg.MODE_EXACT)
        hx.check("host x after the exact host step")
        assert not hagg.touched()
        lib.intsgd_step_host(hg, hx.t, hagg.t, eta_k=0.1, mode=pkg.MODE_FUSED)
        lib.intsgd_get_stats()
        hx.check("host x after the fused host step")
        hagg.check("host aggregate after the fused host step")
        assert hagg.touched()
