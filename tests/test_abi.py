"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2102_08374_b200 as pkg

ROOT = Path(__file__).resolve().parent.parent


def _declared_symbols():
    """Every entry point declared in the public header and in the header of the test / tuning knobs."""
    names = set()
    for header in ("intsgd.h", "intsgd_tuning.h"):
        text = (ROOT / "include" / header).read_text()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(intsgd_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_header_and_binding_list_the_same_entry_points():
    assert _declared_symbols() == sorted(pkg.EXPORTS)


def test_library_builds_loads_and_exports_every_symbol():
    pkg.build()
    lib = ctypes.CDLL(str(pkg.library_path()))
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header():
    from paper_2102_08374_b200 import binding
    assert ctypes.sizeof(binding.Config) == 64
    assert ctypes.sizeof(binding.State) == 32
    assert ctypes.sizeof(binding.Stats) == 32 + 8 * 64 + 8 + 8 + 8


def test_argument_errors_need_no_gpu():
    lib = pkg.load()
    assert lib.intsgd_create(None, None) == pkg.ERR_INVALID_ARG
    assert b"NULL" in lib.intsgd_last_error(None)
    ctx = ctypes.c_void_p()
    from paper_2102_08374_b200.binding import Config
    bad = [dict(n=0), dict(n=65), dict(d=0), dict(grad_dtype=7), dict(payload_dtype=3), dict(rounding=4), dict(rounding=-1),
           dict(beta=1.0), dict(beta=-0.1), dict(eps=-1.0), dict(clip_limit=-5), dict(reserved=1),
           dict(payload_dtype=1, clip_limit=128), dict(n=16, clip_limit=2**28)]
    for kw in bad:
        base = dict(n=4, grad_dtype=0, d=1024, payload_dtype=0, rounding=0, beta=0.9, eps=1e-8, seed=1,
                    clip_limit=0, device=0, reserved=0)
        base.update(kw)
        cfg = Config(**base)
        assert lib.intsgd_create(ctypes.byref(ctx), ctypes.byref(cfg)) == pkg.ERR_INVALID_ARG, kw
        assert not ctx.value
    assert lib.intsgd_scale(None, 0.1, -1.0, None) == pkg.ERR_INVALID_ARG
    assert lib.intsgd_launch_count(None) == 0


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(pkg.IntSGDError) as e:
        pkg.IntSGD(4, 1024)
    assert e.value.code == pkg.ERR_CUDA
