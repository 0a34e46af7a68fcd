"""Mutation pass over the CPU checker: each planted mistake must be caught by the pins.

A mistake is one textual change in a copy of oracle/squant_oracle.c (wrong tie rule, reversed
order, wrong sign, dropped filter, ...).  The copy is compiled into a temporary directory and
swapped in for the checker's library while a battery of pin tests runs; at least one of them must
fail.  This keeps the pins honest: a pin set that a plausible mistake slips through is too weak.
"""
import ctypes
import os
import subprocess

import pytest

import oracle
from oracle import build as oracle_build

import test_oracle_paper_examples as golden
import test_oracle_properties as props
import test_oracle_scales_in as scaled

EKC, EK = oracle.MODE_EKC, oracle.MODE_E | oracle.MODE_K

MUTATIONS = [
    ("half-way flip count goes up", "return (abs_e + SQO_HALF - 1) >> 30;", "return (abs_e + SQO_HALF) >> 30;"),
    ("smaller perturbation first", "return x->mag > y->mag ? -1 : 1;", "return x->mag < y->mag ? -1 : 1;"),
    ("higher index first on ties", "return x->idx < y->idx ? -1 : 1;", "return x->idx > y->idx ? -1 : 1;"),
    ("Over SQuant already at k = |e|", "if (k * SQO_ONE > abs_e) {", "if (k * SQO_ONE >= abs_e) {"),
    ("Over candidate keeps its value from before the flip", "                wk->cv[n] = P[j];\n                wk->cj[n] = j;\n            } else if (k < nc) {",
     "                wk->cv[n] = P[j] + sgn * SQO_ONE;\n                wk->cj[n] = j;\n            } else if (k < nc) {"),
    ("perturbation has the wrong sign", "float p = qf - x;", "float p = x - qf;"),
    ("SQuant-C sums the candidates instead of all elements", "for (int32_t j = 0; j < NK; ++j) ec += P[j];",
     "for (int32_t j = 0; j < n_slots; ++j) ec += wk->cv[j];"),
    ("SQuant-K takes elements of either sign", "if (sqo_sign64(Pk[i]) == sgn && flipped >= qmin && flipped <= qmax) {",
     "if (Pk[i] != 0 && flipped >= qmin && flipped <= qmax) {"),
    ("SQuant-K may flip out of range", "if (sqo_sign64(Pk[i]) == sgn && flipped >= qmin && flipped <= qmax) {",
     "if (sqo_sign64(Pk[i]) == sgn) {"),
    ("qmax is 2^(bits-1)", "const int32_t qmax = (1 << (opt->bits - 1)) - 1;", "const int32_t qmax = (1 << (opt->bits - 1));"),
    ("SQuant-C takes candidates of either sign", "if (sqo_sign64(v) == sgn && flipped >= qmin && flipped <= qmax) {",
     "if (v != 0 && flipped >= qmin && flipped <= qmax) {"),
    ("SQuant-C may flip out of range", "if (sqo_sign64(v) == sgn && flipped >= qmin && flipped <= qmax) {", "if (sqo_sign64(v) == sgn) {"),
    ("SQuant-C flips one kernel too few", "            if (k > nc) k = nc;\n            for (int64_t r = 0; r < k; ++r) {\n                int32_t j = wk->list[r].idx;\n                q[j] -= sgn;\n                P[j] -= sgn * SQO_ONE;\n                wk->flip[j] |= 2;",
     "            if (k > nc) k = nc;\n            for (int64_t r = 1; r < k; ++r) {\n                int32_t j = wk->list[r].idx;\n                q[j] -= sgn;\n                P[j] -= sgn * SQO_ONE;\n                wk->flip[j] |= 2;"),
    ("scale denominator is qmax + 1", "s = (a < 0x1p-100f) ? 1.0f : a / (float)qmax;", "s = (a < 0x1p-100f) ? 1.0f : a / (float)(qmax + 1);"),
    ("supplied scale is ignored", "        s = *scale_in;", "        s = 1.0f; (void)scale_in;"),
    ("clip of Sec. 2.2 is missing at the upper bound", "        if (qf > (float)qmax) qf = (float)qmax;\n", ""),
    ("bfloat16 output is truncated instead of rounded", "    u += 0x7fffu + ((u >> 16) & 1u);\n", ""),
    ("flip count is not limited by the candidates (SQuant-K)", "            int64_t k = sqo_flip_count(abs_e);\n            if (k > nc) k = nc;\n            for (int64_t r = 0; r < k; ++r) {\n                int32_t j = wk->list[r].idx;\n                q[j] -= sgn;\n                P[j] -= sgn * SQO_ONE;\n                wk->flip[j] |= 1;",
     "            int64_t k = sqo_flip_count(abs_e);\n            if (k > nc) k = nc > 0 ? nc - 1 : 0;\n            for (int64_t r = 0; r < k; ++r) {\n                int32_t j = wk->list[r].idx;\n                q[j] -= sgn;\n                P[j] -= sgn * SQO_ONE;\n                wk->flip[j] |= 1;"),
]

# quick pins first; each entry is a call that raises AssertionError when the checker is wrong
BATTERY = (
    [lambda c=c: golden.test_paper_worked_example(c) for c in golden.CASES]
    + [golden.test_three_by_three_needs_at_most_four_flips,
       props.test_half_way_values_round_to_even_and_sign_convention,
       props.test_index_tie_break_is_lowest_flat_index,
       props.test_flip_out_of_range_is_excluded,
       props.test_exactly_integer_kernel_sum_is_under_squant,
       props.test_squant_c_true_channel_sum_not_candidate_sum,
       lambda: props.test_mode_E_is_round_to_nearest((8, 16, 3, 3), 4),
       lambda: props.test_squant_k_is_the_constrained_optimum_bruteforce(4),
       lambda: props.test_squant_k_invariants((8, 16, 3, 3), 4, "coarse"),
       lambda: props.test_squant_c_invariants((8, 16, 3, 3), 4, "coarse"),
       lambda: props.test_squant_c_invariants((2, 300, 1, 1), 8, "normal"),
       lambda: props.test_negation_scaling_permutation((8, 16, 3, 3), EKC),
       lambda: props.test_dequantized_bf16_output_matches_the_library_conversion(4),
       scaled.test_hand_worked_clipped_kernel,
       scaled.test_hand_worked_clipped_channel,
       lambda: scaled.test_supplying_the_absmax_scale_changes_nothing(4, EKC),
       lambda: scaled.test_clipping_invariants((12, 7, 3, 3), 3, EKC),
       lambda: scaled.test_squant_k_with_clipping_is_the_constrained_optimum_bruteforce(4)])


def _killed() -> bool:
    for pin in BATTERY:
        try:
            pin()
        except AssertionError:
            return True
        except Exception:      # a mutant may also crash a pin's own arithmetic (e.g. overflow): that counts
            return True
    return False


def test_the_battery_passes_on_the_real_checker():
    assert not _killed()


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(name, old, new, tmp_path):
    src = open(oracle_build.SRC).read()
    assert src.count(old) >= 1, f"mutation '{name}' no longer applies to the checker's source"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new, 1))
    lib_path = tmp_path / "libmutant.so"
    subprocess.run(["gcc", *oracle_build.CFLAGS, "-o", str(lib_path), str(mutated), "-lm"], check=True)
    real = oracle._load()
    lib = ctypes.CDLL(str(lib_path))
    lib.sqo_quantize_layer_scaled.restype = real.sqo_quantize_layer_scaled.restype
    lib.sqo_quantize_layer_scaled.argtypes = real.sqo_quantize_layer_scaled.argtypes
    oracle._lib = lib
    try:
        assert _killed(), f"planted mistake '{name}' slipped through every pin"
    finally:
        oracle._lib = real
