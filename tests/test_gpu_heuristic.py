"""GPU parity of the heuristic (SwitchML-style) step, Section 5.2 of the IntSGD paper."""
import numpy as np
import pytest
import torch

import oracle
import paper_2102_08374_b200 as pkg
from paper_2102_08374_b200 import synth

from helpers import dev, rel_close, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("grad_dtype,payload_dtype,nb", [(pkg.GRAD_F32, pkg.PAYLOAD_I32, 32), (pkg.GRAD_F32, pkg.PAYLOAD_I8, 8),
                                                         (pkg.GRAD_BF16, pkg.PAYLOAD_I8, 8), (pkg.GRAD_F32, pkg.PAYLOAD_I32, 16)])
def test_heuristic_step_matches_the_oracle(path, grad_dtype, payload_dtype, nb):
    rng = np.random.default_rng(nb + path)
    n, d, eta, seed = 4, 5 * (1 << 15) + 3, 0.1, 9
    x_ref = rng.normal(0, 1, d).astype(np.float32)
    x = to_dev(x_ref.copy())
    agg = torch.zeros(d, dtype=torch.int32, device=dev())
    with pkg.IntSGD(n, d, grad_dtype=grad_dtype, payload_dtype=payload_dtype, seed=seed) as lib:
        lib.intsgd_set_fused_path(path)
        for k in range(3):
            grads = [rng.normal(0, 10.0 ** rng.uniform(-4, 0), d).astype(np.float32) for _ in range(n)]
            grads[1][7] = np.nan                       # ignored by the profiling pass, rounds to 0 and is counted
            if grad_dtype == pkg.GRAD_BF16:
                grads = [synth.to_bf16_bits(g) for g in grads]
            lib.intsgd_heuristic_step([to_dev(g) for g in grads], x, agg, eta_k=eta, num_bits=nb)
            st = lib.intsgd_get_stats()
            mx, e, a, c = oracle.heuristic_scale(grads, n, nb, eta)
            assert st["alpha"] == float(a) and st["c"] == float(c)
            ref = oracle.step_window(grads, x_ref, a, c, step=k, seed=seed, payload_dtype=payload_dtype)
            assert np.array_equal(to_host(agg), ref["agg"])
            assert np.array_equal(to_host(x).view(np.uint32), x_ref.view(np.uint32))
            assert rel_close(st["dx2"], ref["dx2"])
            assert st["clip_count"] == ref["clip_count"] and st["nonfinite"] == ref["nonfinite"] == 1
            assert st["agg_overflow"] == ref["agg_overflow"] and st["max_abs_agg"] == ref["max_abs_agg"]
            assert st["step"] == k + 1 and st["r"] == 0.0
            # the rule's promise: the aggregate fits num_bits
            assert st["max_abs_agg"] <= 2**nb - 1 + n


def test_heuristic_step_without_a_scale_is_reported_and_not_applied():
    d, n = 4099, 2
    x0 = np.arange(d, dtype=np.float32)
    x = to_dev(x0.copy())
    with pkg.IntSGD(n, d) as lib:
        zeros = [torch.zeros(d, device=dev()) for _ in range(n)]
        lib.intsgd_heuristic_step(zeros, x, None, eta_k=0.1, num_bits=8)
        with pytest.raises(pkg.IntSGDError) as e:
            lib.intsgd_get_stats()
        assert e.value.code == pkg.ERR_SCALE_NONFINITE
        inf = [torch.ones(d, device=dev()) for _ in range(n)]
        inf[1][5] = float("inf")
        lib.intsgd_heuristic_step(inf, x, None, eta_k=0.1, num_bits=8)
        assert lib.intsgd_get_stats(allow_nonfinite=True)["status"] == pkg.ERR_SCALE_NONFINITE
        assert np.array_equal(to_host(x), x0)
        for bad in (1, 33):
            with pytest.raises(pkg.IntSGDError) as e:
                lib.intsgd_heuristic_step(zeros, x, None, eta_k=0.1, num_bits=bad)
            assert e.value.code == pkg.ERR_INVALID_ARG
        ones = [torch.ones(d, device=dev()) for _ in range(n)]
        lib.intsgd_heuristic_step(ones, x, None, eta_k=0.1, num_bits=8)      # the context recovers
        st = lib.intsgd_get_stats()
        assert st["status"] == pkg.OK and st["alpha"] == 127.5 and st["step"] == 1
