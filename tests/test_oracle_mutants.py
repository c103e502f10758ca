"""The pins must catch plausible mistakes: each mutant below plants one in a copy of the oracle's
source (on the CPU, in a temporary directory), and the battery of pins has to reject it."""
import ctypes
import subprocess
from pathlib import Path

import pytest

import oracle
import test_oracle_blocks as tb
import test_oracle_compare as tc
import test_oracle_diana as td
import test_oracle_draw16 as t16
import test_oracle_heuristic as th
import test_oracle_philox as tp
import test_oracle_rounding as tr
import test_oracle_scale as ts
import test_oracle_step as tt

SRC = Path(oracle.__file__).resolve().parent / "intsgd_oracle.cpp"
GOLDEN = Path(__file__).resolve().parent / "golden"

# (name, text to find, replacement)
MUTANTS = [
    ("philox multipliers swapped", "constexpr uint32_t kMul0 = 0xD2511F53u;", "constexpr uint32_t kMul0 = 0xCD9E8D57u;"),
    ("philox nine rounds", "for (int round = 0; round < 10; ++round)", "for (int round = 0; round < 9; ++round)"),
    ("philox output words crossed", "const uint32_t n0 = hi1 ^ c1 ^ k0;", "const uint32_t n0 = hi0 ^ c1 ^ k0;"),
    ("philox key schedule dropped", "        k0 += kWeyl0;\n", ""),
    ("counter: worker and step swapped", "(uint32_t)(b >> 32), worker, step}", "(uint32_t)(b >> 32), step, worker}"),
    ("counter: one block per coordinate", "const uint64_t b = j >> 2;", "const uint64_t b = j;"),
    ("uniform keeps 23 bits", "if (len > 24) w &= ~((1u << (len - 24)) - 1u);", "if (len > 23) w &= ~((1u << (len - 23)) - 1u);"),
    ("uniform rounded to nearest, not truncated", "    if (len > 24) w &= ~((1u << (len - 24)) - 1u);", "    "),
    ("draw: a sum on an integer stays down", "return ((double)u >= need) ?", "return ((double)u > need) ?"),
    ("draw: direction reversed", "return ((double)u >= need) ?", "return ((double)u < need) ?"),
    ("draw: complement dropped", "const double need = ((double)k + 1.0) - (double)y;", "const double need = (double)y - (double)k;"),
    ("draw: sum rounded to fp32 before the floor", "return ((double)u >= need) ? (float)((double)k + 1.0) : k;", "return std::floor(y + u);"),
    ("floor replaced by truncation", "const float k = std::floor(y);", "const float k = std::trunc(y);"),
    ("compare form: up iff u <= p", "return f + ((u < p) ? 1.0f : 0.0f);", "return f + ((u <= p) ? 1.0f : 0.0f);"),
    ("compare form: 23-bit draw", "return (float)(w >> 8) * 5.9604644775390625e-8f;", "return (float)(w >> 9) * 5.9604644775390625e-8f;"),
    ("compare form: truncation for floor", "const float f = std::floor(y);", "const float f = std::trunc(y);"),
    ("nearest: ties away from zero", "return std::nearbyintf(y);", "return std::roundf(y);"),
    ("clip: NaN not zeroed", "    if (y != y) qf = 0.0f;\n", ""),
    ("clip: limit off by one", "if (y > Lf) qf = Lf;", "if (y > Lf) qf = Lf + 1.0f;"),
    ("clip count on the rounded value", "r.clipped = !(std::fabs(y) <= Lf);", "r.clipped = !(std::fabs(qf) <= Lf);"),
    ("bf16 widened by 15 bits", "const uint32_t bits = (uint32_t)h << 16;", "const uint32_t bits = (uint32_t)h << 15;"),
    ("scale: (1 - beta) dropped", "const double b = (1.0 - beta) * dx2;\n    const double r = a + b;\n    const double num = std::sqrt((double)d);",
     "const double b = dx2;\n    const double r = a + b;\n    const double num = std::sqrt((double)d);"),
    ("scale: n instead of 2n", "const double two_n_r = (2.0 * (double)n) * r;\n    const double eta2", "const double two_n_r = ((double)n) * r;\n    const double eta2"),
    ("scale: eps not squared", "const double eps2 = eps * eps;", "const double eps2 = eps;"),
    ("scale: eta not squared", "const double eta2 = eta * eta;", "const double eta2 = eta;"),
    ("scale: c uses 1/alpha only", "const float c = (float)(eta / ((double)n * (double)alpha));\n    *r_out = r;\n    *alpha64_out = alpha64;\n    *alpha_out = alpha;\n    *c_out = c;\n}\n\n// Algorithm 2",
     "const float c = (float)(eta / ((double)alpha));\n    *r_out = r;\n    *alpha64_out = alpha64;\n    *alpha_out = alpha;\n    *c_out = c;\n}\n\n// Algorithm 2"),
    ("block scale: sqrt(d) instead of sqrt(d_l)", "const double num = eta * std::sqrt((double)d_l);", "const double num = eta * std::sqrt((double)d);"),
    ("block scale: guard not shared", "const double share = (double)d_l / (double)d;", "const double share = 1.0;"),
    ("aggregate: update sign", "const float x_new = x_old - t;\n        const float dj = x_new - x_old;\n        dx2 += (double)dj * (double)dj;\n        x[j] = x_new;\n    }\n    *dx2_out = dx2;\n}\n\n// ---- Algorithm 1, Init",
     "const float x_new = x_old + t;\n        const float dj = x_new - x_old;\n        dx2 += (double)dj * (double)dj;\n        x[j] = x_new;\n    }\n    *dx2_out = dx2;\n}\n\n// ---- Algorithm 1, Init"),
    ("aggregate: one worker skipped", "for (int32_t i = 0; i < n; ++i) {\n            S += (payload_dtype == 1)", "for (int32_t i = 1; i < n; ++i) {\n            S += (payload_dtype == 1)"),
    ("exact step: eta not divided by n", "const float c0 = (float)(eta / (double)n);", "const float c0 = (float)(eta);"),
    ("sqdiff: difference not squared", "s += (double)dj * (double)dj;", "s += (double)dj;"),
    ("diana: shift moved by the raw integer", "const float dq = ainv * (float)r.q;", "const float dq = (float)r.q;"),
    ("diana: estimator without the shift", "const float gt = h_global[t] + dec;", "const float gt = dec;"),
    ("16-bit draws: halves swapped", "const uint32_t v = (e & 1) ? (word >> 16) : (word & 0xFFFFu);", "const uint32_t v = (e & 1) ? (word & 0xFFFFu) : (word >> 16);"),
    ("16-bit draws: wrong word of the pair", "const uint32_t word = out[2 * h + (e >> 1)];", "const uint32_t word = out[h + (e >> 1)];"),
    ("16-bit draws: partner at distance 256", "const uint32_t h = (uint32_t)((u >> 9) & 1);", "const uint32_t h = (uint32_t)((u >> 8) & 1);"),
    ("heuristic: exponent rounded down", "const int max_exp = (m == 0.5f) ? e - 1 : e;", "const int max_exp = e - 1;"),
]


def _build(tmp_path, idx, text):
    src = tmp_path / f"mutant_{idx}.cpp"
    so = tmp_path / f"mutant_{idx}.so"
    src.write_text(text)
    subprocess.run(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC", "-o", str(so),
                    str(src)], check=True)
    return oracle._declare(ctypes.CDLL(str(so)))


def _battery():
    """A compact selection of the pins; raises AssertionError on the first one that fails."""
    tp.test_known_answer_vectors(GOLDEN)
    tp.test_stream_layout()
    tp.test_uniform_from_word_is_the_word_truncated_to_fp32()
    tr.test_int_definition_against_exact_rationals()
    tr.test_negative_half_integers()
    tr.test_floor_of_the_unrounded_sum_on_adversarial_values()
    tr.test_unbiased_and_variance_monte_carlo(0.25)
    tr.test_nearest_even()
    tr.test_clip_counts_closed_form_int8()
    tr.test_clip_is_independent_of_the_draw_and_keeps_values_in_range()
    tr.test_default_int32_limit_makes_the_sum_fit()
    tr.test_non_finite_values_on_the_int32_wire()
    ts.test_hand_example(GOLDEN)
    ts.test_closed_form_invariant_and_unrolled_average()
    ts.test_block_rule_closed_form()
    ts.test_algorithm_2_with_one_block_equals_algorithm_1()
    ts.test_safeguard_regimes()
    tt.test_hand_example(GOLDEN)
    tt.test_exact_first_step_is_mean_gradient_axpy()
    tt.test_sqdiff_and_dx2_agree_with_numpy_fp64()
    tt.test_windows_reproduce_the_full_vector()
    tt.test_bf16_gradients_are_widened_exactly()
    tt.test_int8_aggregate_overflow_count_and_max()
    td.test_hand_example(GOLDEN)
    td.test_zero_shifts_give_the_intsgd_integers_and_step()
    th.test_hand_values()
    t16.test_layout_against_an_independent_statement()
    tc.test_uniform24_is_the_top_24_bits()
    tc.test_definition_against_exact_rationals()
    tc.test_half_integers_and_boundaries()


def test_the_unmodified_oracle_passes_the_battery(tmp_path, monkeypatch):
    monkeypatch.setattr(oracle, "_lib", _build(tmp_path, "clean", SRC.read_text()))
    _battery()


@pytest.mark.parametrize("idx", range(len(MUTANTS)), ids=[m[0] for m in MUTANTS])
def test_every_planted_mistake_is_caught(idx, tmp_path, monkeypatch):
    name, find, repl = MUTANTS[idx]
    text = SRC.read_text()
    assert text.count(find) >= 1, f"mutation site not found: {name}"
    monkeypatch.setattr(oracle, "_lib", _build(tmp_path, idx, text.replace(find, repl, 1)))
    with pytest.raises((AssertionError, Exception)) as caught:
        _battery()
    assert caught.type is not None
