"""Shows that the pins have teeth: each plausible mistake, planted in a COPY of the oracle's C
source on the CPU, must make at least one pin test fail.  (The real oracle is never modified.)"""
import os
import subprocess

import pytest

import test_oracle_pins as pins
import test_oracle_bias_and_packing_pins as bpins
import test_oracle_two_breakpoints_pins as tpins
import test_oracle_three_breakpoints_pins as t3pins
import test_oracle_unsigned_pins as upins

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "pwlq_oracle.c")

MUTANTS = {
    "tail_closed_at_p": ("int tail = (a > p);", "int tail = (a >= p);"),
    "round_half_away": ("fminf(rintf(t), P->Lf)", "fminf(roundf(t), P->Lf)"),
    "truncate": ("fminf(rintf(t), P->Lf)", "fminf(floorf(t), P->Lf)"),
    "levels_2^(b-1)": ("P.Lf = (float)((1 << (bits - 1)) - 1);", "P.Lf = (float)(1 << (bits - 1));"),
    "levels_b_bits": ("P.Lf = (float)((1 << (bits - 1)) - 1);", "P.Lf = (float)((1 << bits) - 1);"),
    "drop_offset": ("    v = v + z;                             /* ... + z, Eq. 1 first line         */",
                    "    v = v + 0.0f;"),
    "offset_not_subtracted": ("float u = a - z;", "float u = a;"),
    "tail_range_is_m": ("d = m - p;", "d = m;"),
    "swap_steps": ("float s = tail ? P->s2 : P->s1;", "float s = tail ? P->s1 : P->s2;"),
    "swap_inverses": ("float inv = tail ? P->inv2 : P->inv1;", "float inv = tail ? P->inv1 : P->inv2;"),
    "sign_from_leq": ("neg = (x[i] < 0.0f);", "neg = (x[i] <= 0.0f);"),
    "sign_bit_position": ("code = (neg << (bits - 1)) | q;\n            y = neg",
                          "code = (neg << bits) | q;\n            y = neg"),
    "mask_bit_order": ("region_mask[i >> 3] |= (uint8_t)(1u << (i & 7));",
                       "region_mask[i >> 3] |= (uint8_t)(0x80u >> (i & 7));"),
    "nibble_order": ("codes[i >> 1] |= (uint8_t)(code << ((i & 1) * 4));",
                     "codes[i >> 1] |= (uint8_t)(code << ((1 - (i & 1)) * 4));"),
    "argmin_last_on_ties": ("if (k == 0 || sse < best)", "if (k == 0 || sse <= best)"),
    "argmax": ("if (k == 0 || sse < best)", "if (k == 0 || sse > best)"),
    "abs_error_not_squared": ("sse += d * d;", "sse += fabs(d);"),
    "absmax_signed": ("float a = fabsf(x[i]);\n            if (!(a <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;\n            if (a > m) m = a;\n        }\n        m_out[c] = m;",
                      "float a = x[i];\n            if (!(a <= 3.402823466e+38f)) return ORACLE_ERR_NONFINITE;\n            if (a > m) m = a;\n        }\n        m_out[c] = m;"),
    "dequant_ignores_region": ("float z = r ? p : 0.0f;\n            float v = q * s;", "float z = 0.0f;\n            float v = q * s;"),
    "p_from_wrong_ratio": ("float p = m * ratios[k];", "float p = m * ratios[K - 1 - k];"),
    "eq9_wrong_sign": ("- (2.0 * m - p + m * (m - 2.0 * p) * model_pdf(model, scale, p));",
                       "- (2.0 * m - p - m * (m - 2.0 * p) * model_pdf(model, scale, p));"),
    "eq9_dropped_p": ("- (2.0 * m - p + m", "- (2.0 * m + m"),
    "sigma_without_sqrt": (": sqrt(s2 / (double)(e - b));", ": (s2 / (double)(e - b));"),
    "laplace_cdf_as_gauss_tail": ("return 1.0 - 0.5 * exp(-p / scale);", "return 1.0 - exp(-p / scale);"),
    "approx_constant": ("0.8614 * (m / scale) + 0.6079", "0.8614 * (m / scale) + 0.06079"),
    "unsigned_levels_as_signed": ("return make_params(m, p, bits + 1);", "return make_params(m, p, bits);"),
    "unsigned_no_shift": ("    float a = x - lo;\n    a = fmaxf(a, 0.0f);", "    float a = x;\n    a = fmaxf(a, 0.0f);"),
    "unsigned_no_clamp_below": ("    a = fmaxf(a, 0.0f);", "    a = a + 0.0f;"),
    "unsigned_offset_not_added": ("if (fake_out) fake_out[i] = v + lo;", "if (fake_out) fake_out[i] = v;"),
    "unsigned_dequant_offset": ("            y[i] = v + lo;", "            y[i] = v;"),
    "unsigned_dequant_level_mask": ("int qmask = (1 << bits) - 1;", "int qmask = (1 << (bits - 1)) - 1;"),
    "minmax_min_is_max": ("if (i == b || x[i] < lo) lo = x[i];", "if (i == b || x[i] > lo) lo = x[i];"),
    "unsigned_range_is_hi": ("        float m = hi_in[c] - lo;\n        double best = 0.0;", "        float m = hi_in[c];\n        double best = 0.0;"),
    "two_bp_region_closed_at_p1": ("int r = (a > p1) + (a > p2);", "int r = (a >= p1) + (a > p2);"),
    "two_bp_middle_range": ("d[0] = p1; d[1] = p2 - p1; d[2] = m - p2;", "d[0] = p1; d[1] = p2; d[2] = m - p2;"),
    "two_bp_third_offset": ("P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2;", "P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p1;"),
    "two_bp_last_pair_on_ties": ("if (i < j && (first || sse < best))", "if (i < j && (first || sse <= best))"),
    "two_bp_region_bit_order": ("region2[i >> 2] |= (uint8_t)(r << ((i & 3) * 2));",
                                "region2[i >> 2] |= (uint8_t)(r << ((3 - (i & 3)) * 2));"),
    "two_bp_pairs_not_ordered": ("if (i < j && m > 0.0f) {", "if (i != j && m > 0.0f) {"),
    "three_bp_region_closed_at_p3": ("int r = (a > P->z[1]) + (a > P->z[2]) + (a > P->z[3]);",
                                     "int r = (a > P->z[1]) + (a > P->z[2]) + (a >= P->z[3]);"),
    "three_bp_third_range": ("d[0] = p1; d[1] = p2 - p1; d[2] = p3 - p2; d[3] = m - p3;",
                             "d[0] = p1; d[1] = p2 - p1; d[2] = p3 - p1; d[3] = m - p3;"),
    "three_bp_fourth_offset": ("P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2; P.z[3] = p3;",
                               "P.z[0] = 0.0f; P.z[1] = p1; P.z[2] = p2; P.z[3] = p2;"),
    "three_bp_last_triple_on_ties": ("if (valid && (first || sse < best))",
                                     "if (valid && (first || sse <= best))"),
    "three_bp_triples_not_ordered": ("int valid = (i < j && j < k);", "int valid = (i < j && i < k && j != k);"),
    "three_bp_breakpoints_swapped": ("make_params3(m, m * ratios[i], m * ratios[j], m * ratios[k], bits);",
                                     "make_params3(m, m * ratios[i], m * ratios[k], m * ratios[j], bits);"),
    "three_bp_dequant_region_capped": ("            float v = q * P.s[r];\n            v = v + P.z[r];\n            if (!(m > 0.0f)) { v = 0.0f; neg = 0; }\n            y[i] = neg ? -v : v;\n        }\n    }\n    return ORACLE_OK;\n}\n\n/* ------------------------------------------------------------------------------------------\n * Bias",
                                       "            float v = q * P.s[r > 2 ? 2 : r];\n            v = v + P.z[r > 2 ? 2 : r];\n            if (!(m > 0.0f)) { v = 0.0f; neg = 0; }\n            y[i] = neg ? -v : v;\n        }\n    }\n    return ORACLE_OK;\n}\n\n/* ------------------------------------------------------------------------------------------\n * Bias"),
    "bc_ratio_inverted": ("xi = sqrt(vx / vy);", "xi = sqrt(vy / vx);"),
    "bc_variance_ratio_without_sqrt": ("xi = sqrt(vx / vy);", "xi = (vx / vy);"),
    "bc_offset_sign": ("beta_out[c] = (float)(mx - xi * my);", "beta_out[c] = (float)(mx + xi * my);"),
    "bc_offset_before_scale": ("            float t = xi_in[c] * y[i];\n            y[i] = t + beta_in[c];",
                               "            float t = y[i] + beta_in[c];\n            y[i] = xi_in[c] * t;"),
    "dense_region_in_low_bit": ("int field = (codes_u8[i] & ((1 << bits) - 1)) | (r << bits);",
                                "int field = ((codes_u8[i] & ((1 << bits) - 1)) << 1) | r;"),
    "dense_msb_first": ("if ((field >> k) & 1) stream[pos >> 3] |= (uint8_t)(1u << (pos & 7));",
                        "if ((field >> k) & 1) stream[pos >> 3] |= (uint8_t)(0x80u >> (pos & 7));"),
    "divide_not_reciprocal_free_pass": None,   # placeholder documented below
}
# 'divide_not_reciprocal': evaluating (|r| - z) / s by a true division instead of multiplying by
# fl(L / Delta) is a different but equally valid reading of Eq. 1; it changes levels only at
# binary32-noise distance from a tie, which no pin can (or should) tell apart.
del MUTANTS["divide_not_reciprocal_free_pass"]

PIN_CALLS = [
    lambda o: pins.test_worked_example_b3(o),
    lambda o: pins.test_absmax_rows_and_sign(o),
    lambda o: pins.test_params_step_is_range_over_levels(o, 4),
    lambda o: pins.test_levels_regions_and_half_step_bound(o, 4),
    lambda o: pins.test_p_equals_m_is_symmetric_uniform(o, 4),
    lambda o: pins.test_bruteforce_dense_grid_tiny_rows(o, 3, 32),
    lambda o: pins.test_lowest_index_wins_ties(o),
    lambda o: pins.test_zero_rows_and_single_values(o),
    lambda o: pins.test_ragged_rows_equal_dense_rows(o),
    lambda o: pins.test_uniform_data_matches_eq2(o),
    lambda o: pins.test_analytic_root_matches_an_independent_solver(o, 1, pins.stats.norm),
    lambda o: pins.test_analytic_root_matches_an_independent_solver(o, 2, pins.stats.laplace),
    lambda o: pins.test_analytic_approximation_and_scales(o),
    lambda o: upins.test_worked_example_unsigned_b2(o),
    lambda o: upins.test_minmax_rows(o),
    lambda o: upins.test_nonnegative_rows_equal_the_signed_scheme_with_one_more_bit(o, 3),
    lambda o: upins.test_levels_regions_and_half_step_bound_unsigned(o, 4),
    lambda o: upins.test_bruteforce_true_division_tiny_rows(o, 4, 32),
    lambda o: tpins.test_worked_example_two_breakpoints(o),
    lambda o: tpins.test_second_breakpoint_at_m_is_the_one_breakpoint_scheme(o, 3),
    lambda o: tpins.test_pair_order_and_degenerate_rows(o),
    lambda o: tpins.test_half_step_bound_per_region(o, 4),
    lambda o: t3pins.test_worked_example_three_breakpoints(o),
    lambda o: t3pins.test_third_breakpoint_at_m_is_the_two_breakpoint_scheme(o, 3),
    lambda o: t3pins.test_triple_order_and_degenerate_rows(o),
    lambda o: t3pins.test_half_step_bound_per_region_three_breakpoints(o, 4),
    lambda o: bpins.test_corrected_rows_keep_mean_and_centred_norm(o, 4),
    lambda o: bpins.test_hand_computed_row(o),
    lambda o: bpins.test_dequantize_with_correction_applies_scale_then_offset(o),
    lambda o: bpins.test_dense_stream_hand_example(o),
]


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path, oracle):
    old, new = MUTANTS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation site for {name} not found"
    mutated = tmp_path / "mutant.c"
    mutated.write_text(src.replace(old, new))
    so = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-o", str(so),
                    str(mutated), "-lm"], check=True)
    mutant = oracle.OracleLib(str(so))
    caught = []
    for i, call in enumerate(PIN_CALLS):
        try:
            call(mutant)
        except (AssertionError, oracle.OracleError):
            caught.append(i)
    assert caught, f"no pin noticed the planted mistake '{name}'"
