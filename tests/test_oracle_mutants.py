"""Tests of the pins themselves.  Each case plants one plausible mistake in a COPY of the oracle's C
source (a dropped term, a wrong sign or index, a transposed operand, a wrong rounding), builds it, and
requires that at least one pin of test_oracle_pins.py fails against it.  Everything runs on the CPU."""
import os

import pytest

import oracle
import test_oracle_asym_pins as apins
import test_oracle_pins as pins
import test_oracle_search_pins as spins
import test_oracle_int4_pins as ipins

SRC = open(os.path.join(os.path.dirname(oracle.__file__), "ptq_oracle.c")).read()

# (name, text to find, replacement, pins expected to notice)
MUTANTS = [
    ("truncate instead of round-to-nearest", "r = nearbyintf(v);", "r = truncf(v);",
     [lambda: pins.test_quantizer_ties_clamp_and_specials()]),
    ("ties away from zero", "r = nearbyintf(v);", "r = roundf(v);",
     [lambda: pins.test_quantizer_ties_clamp_and_specials()]),
    ("clamp to the symmetric range", "if (r < -128.0f) r = -128.0f;", "if (r < -127.0f) r = -127.0f;",
     [lambda: pins.test_quantizer_ties_clamp_and_specials()]),
    ("NaN not mapped to zero", "if (isnan(v)) return 0;", "if (isnan(v)) return 127;",
     [lambda: pins.test_quantizer_ties_clamp_and_specials()]),
    ("multiply by s instead of dividing", "volatile float u = xf / s;", "volatile float u = xf * s;",
     [lambda: pins.test_quantizer_indexes_token_position_and_channel()]),
    ("one fused division", "volatile float v = u / dx;", "volatile float v = xf / (s * dx);",
     [lambda: pins.test_quantizer_keeps_the_two_divisions_separate()]),
    ("reciprocal multiplications instead of divisions", "volatile float u = xf / s;\n    volatile float v = u / dx;",
     "volatile float rs_ = 1.0f / s; volatile float rd_ = 1.0f / dx; volatile float u = xf * rs_;\n    volatile float v = u * rd_;",
     [lambda: pins.test_quantizer_keeps_the_two_divisions_separate()]),
    ("step indexed by row instead of token position", "q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[k], dx[t]);",
     "q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[k], dx[m % 2]);",
     [lambda: pins.test_quantizer_indexes_token_position_and_channel()]),
    ("smoothing scale of the wrong channel", "q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[k], dx[t]);",
     "q[m * K + k] = ptqo_quantize_one(x[m * K + k], s[(k + 1) % K], dx[t]);",
     [lambda: pins.test_quantizer_indexes_token_position_and_channel()]),
    ("transposed weight in the contraction", "sum += (int64_t)q[m * K + k] * (int64_t)wq[(long)n * K + k];\n            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;\n            acc[m * N + n]",
     "sum += (int64_t)q[m * K + k] * (int64_t)wq[((long)k * N + n) % ((long)N * K)];\n            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;\n            acc[m * N + n]",
     [lambda: pins.test_int_matmul_brute_force_tiny()]),
    ("last term of the contraction dropped", "for (k = 0; k < K; ++k)\n                sum += (int64_t)q[m * K + k] * (int64_t)wq[(long)n * K + k];\n            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;\n            acc[m * N + n]",
     "for (k = 0; k + 1 < K; ++k)\n                sum += (int64_t)q[m * K + k] * (int64_t)wq[(long)n * K + k];\n            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;\n            acc[m * N + n]",
     [lambda: pins.test_int_matmul_one_hot_and_extremes()]),
    ("dequant forgets the activation step", "double yd = (double)acc[m * N + n] * (double)dx[t] * (double)dw[n];",
     "double yd = (double)acc[m * N + n] * (double)dw[n];",
     [lambda: pins.test_dequant_power_of_two_steps_exact()]),
    ("dequant uses the weight step of the row", "double yd = (double)acc[m * N + n] * (double)dx[t] * (double)dw[n];",
     "double yd = (double)acc[m * N + n] * (double)dx[t] * (double)dw[m % N];",
     [lambda: pins.test_dequant_power_of_two_steps_exact()]),
    ("bias subtracted", "if (bias) yd += (double)bias[n];\n            y[m * N + n]", "if (bias) yd -= (double)bias[n];\n            y[m * N + n]",
     [lambda: pins.test_dequant_equals_product_of_dequantized_operands()]),
    ("half conversion rounds toward zero", "double m = nearbyint(ldexp(f, 11));", "double m = floor(ldexp(f, 11));",
     [lambda: pins.test_double_to_half_roundtrip_and_midpoints()]),
    ("overflow saturates to the largest half", "if (a >= 65520.0) return (uint16_t)(sign | 0x7c00);",
     "if (a >= 65520.0) return (uint16_t)(sign | 0x7bff);",
     [lambda: pins.test_double_to_half_roundtrip_and_midpoints()]),
    ("subnormal halves decoded with the wrong scale", "v = ldexpf((float)frac, -24);", "v = ldexpf((float)frac, -25);",
     [lambda: pins.test_half_to_float_all_patterns()]),
    ("fused forward drops the bias", "if (bias) yd += (double)bias[n];\n            y[(m - m0) * N + n]",
     "y[(m - m0) * N + n]", [lambda: pins.test_forward_rows_equals_composition_and_row_ranges()]),
    ("fused forward ignores the row offset", "y[(m - m0) * N + n] = ptqo_double_to_half(yd);",
     "y[((m - m0) * N + n + 1) % ((m1 - m0) * N)] = ptqo_double_to_half(yd);",
     [lambda: pins.test_forward_rows_equals_composition_and_row_ranges()]),
    ("smoothing scale without the square root", "s[k] = sqrtf(ratio);", "s[k] = ratio;",
     [lambda: pins.test_calibrate_vs_numpy_float32_and_no_clip_invariant()]),
    ("calibration divides by 128", "volatile float d = mu / 127.0f;", "volatile float d = mu / 128.0f;",
     [lambda: pins.test_calibrate_vs_numpy_float32_and_no_clip_invariant()]),
    ("weight magnitude ignores the weight step", "volatile float a = fabsf((float)wq[(long)n * K + k]) * dw[n];",
     "volatile float a = fabsf((float)wq[(long)n * K + k]);",
     [lambda: pins.test_calibrate_degenerate_channels_and_positions()]),
    ("calibration without the floor", "if (mu < floor_) mu = floor_;", "",
     [lambda: pins.test_calibrate_degenerate_channels_and_positions()]),
    ("per-tensor step from the raw activations", "volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];\n            float a = fabsf(u);\n            if (a > mu) mu = a;\n        }\n    if (mu < floor_) mu = floor_;",
     "volatile float u = ptqo_half_to_float(xcal[m * K + k]);\n            float a = fabsf(u);\n            if (a > mu) mu = a;\n        }\n    if (mu < floor_) mu = floor_;",
     [lambda: pins.test_calibrate_per_tensor_vs_numpy_float32_and_invariants()]),
    ("per-tensor step over 128 levels", "volatile float d = mu / 127.0f;\n        *delta = d;", "volatile float d = mu / 128.0f;\n        *delta = d;",
     [lambda: pins.test_calibrate_per_tensor_vs_numpy_float32_and_invariants()]),
    ("per-tensor step of the last position only", "    for (m = 0; m < M; ++m)\n        for (k = 0; k < K; ++k) {\n            volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];\n            float a = fabsf(u);\n            if (a > mu) mu = a;",
     "    for (m = T - 1; m < M; m += T)\n        for (k = 0; k < K; ++k) {\n            volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];\n            float a = fabsf(u);\n            if (a > mu) mu = a;",
     [lambda: pins.test_calibrate_per_tensor_vs_numpy_float32_and_invariants()]),
    ("search: error with the wrong sign of the dequantized value", "e = fmaf(-delta, r, u);", "e = fmaf(delta, r, u);",
     [lambda: spins.test_search_zero_loss_on_grid_points_and_ties_keep_the_largest_ratio()]),
    ("search: L1 instead of L2 loss", "acc += (double)e * (double)e;", "acc += fabs((double)e);",
     [lambda: spins.test_search_loss_follows_the_uniform_rounding_error_law()]),
    ("search: codes not clipped", "if (r < -128.0f) r = -128.0f;\n                    e = fmaf", "e = fmaf",
     [lambda: spins.test_search_truncates_when_an_outlier_stretches_the_range()]),
    ("search: ties go to the smallest ratio", "if (j == n_grid || acc < best_loss) {", "if (j == n_grid || acc <= best_loss) {",
     [lambda: spins.test_search_zero_loss_on_grid_points_and_ties_keep_the_largest_ratio()]),
    ("search: candidate grid shifted by one", "volatile float ratio = (float)j / (float)n_grid;\n            volatile float delta = base[t] * ratio;\n            double acc",
     "volatile float ratio = (float)(j - 1) / (float)n_grid;\n            volatile float delta = base[t] * ratio;\n            double acc",
     [lambda: spins.test_search_matches_exact_rational_brute_force()]),
    ("search: non-finite activations poison the loss", "if (!isfinite(u)) continue;", "",
     [lambda: spins.test_search_skips_non_finite_values_and_uses_the_pinned_quantizer()]),
    ("search: largest loss chosen", "if (j == n_grid || acc < best_loss) {", "if (j == n_grid || acc > best_loss) {",
     [lambda: spins.test_search_truncates_when_an_outlier_stretches_the_range()]),
    ("search: smoothing scale ignored", "volatile float u = ptqo_half_to_float(xcal[m * K + k]) / s[k];\n                    volatile float v;",
     "volatile float u = ptqo_half_to_float(xcal[m * K + k]);\n                    volatile float v;",
     [lambda: spins.test_search_matches_exact_rational_brute_force()]),
    ("search: returned step is the full step", "volatile float ratio = (float)best_j / (float)n_grid;", "volatile float ratio = 1.0f;",
     [lambda: spins.test_search_truncates_when_an_outlier_stretches_the_range()]),
    ("int4: nibbles swapped when packing", "packed[r * pb + i] = (uint8_t)(((hi << 4) | (lo & 15)) & 0xff);",
     "packed[r * pb + i] = (uint8_t)(((lo << 4) | (hi & 15)) & 0xff);",
     [lambda: ipins.test_pack_matches_the_hand_evaluated_bytes()]),
    ("int4: low nibble not masked", "packed[r * pb + i] = (uint8_t)(((hi << 4) | (lo & 15)) & 0xff);",
     "packed[r * pb + i] = (uint8_t)(((hi << 4) | lo) & 0xff);",
     [lambda: ipins.test_pack_matches_the_hand_evaluated_bytes()]),
    ("int4: unpack without sign extension", "d[r * cols + k] = (int8_t)(nib >= 8 ? nib - 16 : nib);", "d[r * cols + k] = (int8_t)nib;",
     [lambda: ipins.test_pack_round_trip_all_pairs_and_odd_lengths()]),
    ("int4: unpack reads the wrong nibble", "int nib = (packed[r * pb + k / 2] >> ((k & 1) * 4)) & 15;",
     "int nib = (packed[r * pb + k / 2] >> (((k & 1) ^ 1) * 4)) & 15;",
     [lambda: ipins.test_pack_round_trip_all_pairs_and_odd_lengths()]),
    ("int4: symmetric clamp", "if (r < -8.0f) r = -8.0f;", "if (r < -7.0f) r = -7.0f;",
     [lambda: ipins.test_quantize4_is_the_clipped_eight_bit_code_and_matches_numpy()]),
    ("int4: eight-bit clamp left in", "if (r > 7.0f) r = 7.0f;", "if (r > 127.0f) r = 127.0f;",
     [lambda: ipins.test_quantize4_is_the_clipped_eight_bit_code_and_matches_numpy()]),
    ("int4: step over 8 levels", "volatile float d = mu / 7.0f;", "volatile float d = mu / 8.0f;",
     [lambda: ipins.test_calibrate4_steps_and_no_clip_invariant()]),
    ("dynamic step from the raw activations", "volatile float u = ptqo_half_to_float(x[m * K + k]) / s[k];\n            float a = fabsf(u);\n            if (a > mu) mu = a;                 /* NaN never wins the comparison */",
     "volatile float u = ptqo_half_to_float(x[m * K + k]);\n            float a = fabsf(u);\n            if (a > mu) mu = a;",
     [lambda: pins.test_dynamic_quantizer_vs_numpy_and_invariants()]),
    ("dynamic step over 128 levels", "volatile float d = mu / 127.0f;\n            dx_row[m] = d;", "volatile float d = mu / 128.0f;\n            dx_row[m] = d;",
     [lambda: pins.test_dynamic_quantizer_vs_numpy_and_invariants()]),
    ("zero offset subtracted instead of added", "r = (double)nearbyintf(v) + (double)z;", "r = (double)nearbyintf(v) - (double)z;",
     [lambda: apins.test_asym_indices_ties_and_clamp()]),
    ("offset added before rounding", "r = (double)nearbyintf(v) + (double)z;", "r = (double)nearbyintf(v + (float)z);",
     [lambda: apins.test_asym_indices_ties_and_clamp()]),
    ("contraction keeps the offset", "sum += ((int64_t)c[m * K + k] - (int64_t)z[t]) * (int64_t)wq[(long)n * K + k];",
     "sum += ((int64_t)c[m * K + k]) * (int64_t)wq[(long)n * K + k];",
     [lambda: apins.test_asym_matmul_brute_force_and_closed_form()]),
    ("asymmetric step over 256 levels", "d = range / 255.0f;", "d = range / 256.0f;",
     [lambda: apins.test_asym_calibration_vs_numpy_and_never_clips()]),
    ("zero offset truncated", "r = nearbyintf(zr);", "r = floorf(zr);",
     [lambda: apins.test_asym_calibration_vs_numpy_and_never_clips()]),
    ("range does not include zero", "float lo = 0.0f, hi = 0.0f;", "float lo = 1e30f, hi = -1e30f;",
     [lambda: apins.test_asym_calibration_range_contains_zero_and_degenerate_positions()]),
]


@pytest.mark.parametrize("name,find,repl,checks", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught_by_a_pin(tmp_path, name, find, repl, checks):
    assert SRC.count(find) >= 1, "mutation site not found: %s" % name
    with oracle.use_library(SRC.replace(find, repl, 1), str(tmp_path)):      # the first occurrence only
        caught = 0
        for check in checks:
            try:
                check()
            except AssertionError:
                caught += 1
            except OverflowError:
                caught += 1
        assert caught >= 1, "no pin noticed: %s" % name
    # and the unmodified oracle passes the same checks
    for check in checks:
        check()
