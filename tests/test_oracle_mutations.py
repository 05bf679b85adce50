"""The pins must be able to fail: each case plants one plausible mistake in a copy of the oracle's
C source (on the CPU, in a temporary directory), builds it, and checks that the pin suite rejects it."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "segquant_oracle.c")

MUTATIONS = {
    "ties_away_from_zero": ("static float rne(float v) { return nearbyintf(v); }",
                            "static float rne(float v) { return roundf(v); }"),
    "pos_scale_uses_neg_range": ("s_pos[p] = hi > 0.0f ? hi / q_max : 1.0f;",
                                 "s_pos[p] = hi > 0.0f ? hi / q_min_abs : 1.0f;"),
    "neg_clamp_uses_pos_range": ("clampf(rne(v), -q_min_abs, 0.0f)", "clampf(rne(v), -q_max, 0.0f)"),
    "polarity_test_flipped": ("} else if (x >= 0.0f) {\n                float v = x / s_pos[p];\n                c_pos[m * ldc + k] = (int8_t)",
                              "} else if (x <= 0.0f) {\n                float v = x / s_pos[p];\n                c_pos[m * ldc + k] = (int8_t)"),
    "weight_scale_index_transposed": ("double sw = (double)s_w[p * Q + q];", "double sw = (double)s_w[q * P + p];"),
    "negative_path_dropped": ("v += u; av += fabs(u);", "av += fabs(u);"),
    "negative_path_subtracted": ("v += u; av += fabs(u);", "v -= u; av += fabs(u);"),
    "segment_off_by_one": ("for (int64_t k = kb[p]; k < kb[p + 1]; k++)\n                    s += (int64_t)Xq",
                           "for (int64_t k = kb[p] + 1; k < kb[p + 1]; k++)\n                    s += (int64_t)Xq"),
    "weight_operand_transposed": ("(int64_t)Wq[n * ldw + k]", "(int64_t)Wq[k * ldw + n]"),
    "bias_dropped": ("if (bias) { v += (double)bias[n];", "if (bias) { v += 0.0;"),
    "e4m3_no_mantissa_carry": ("if (q == 8) { q = 0; ex += 1; }\n        int code", "if (q == 8) { q = 7; }\n        int code"),
    "e4m3_subnormals_flushed": ("mag = (uint8_t)nearbyint(ldexp(a, 9));", "mag = 0;"),
    "segment_lookup_off": ("while (s + 1 < nseg && i >= bounds[s + 1]) s++;", "while (s + 1 < nseg && i > bounds[s + 1]) s++;"),
    "e4m3_weight_scale_index_transposed": (
        "float v = W[n * ld + k] / s_w[p * Q + q];\n            Wq[n * ldq + k] = sqo_e4m3_encode(",
        "float v = W[n * ld + k] / s_w[q * P + p];\n            Wq[n * ldq + k] = sqo_e4m3_encode("),
    "i8_weight_scale_index_transposed": (
        "float v = W[n * ld + k] / s_w[p * Q + q];\n            Wq[n * ldq + k] = (int8_t)",
        "float v = W[n * ld + k] / s_w[q * P + p];\n            Wq[n * ldq + k] = (int8_t)"),
    "e4m3_single_scale_clamped_to_positive": ("sqo_e4m3_encode(clampf(x / s_pos[p], -448.0f, 448.0f))",
                                              "sqo_e4m3_encode(clampf(x / s_pos[p], 0.0f, 448.0f))"),
    "abs_sum_doubled": ("v += t; av += fabs(t);", "v += t; av += 2.0 * fabs(t);"),
    "abs_sum_misses_bias": ("av += fabs((double)bias[n]); }", "}"),
    "abs_sum_misses_negative_path": ("v += u; av += fabs(u);", "v += u;"),
    "e4m3_weight_not_clipped": ("sqo_e4m3_encode(clampf(v, -448.0f, 448.0f))", "sqo_e4m3_encode(v * 0.5f)"),
    "asym_zero_point_wrong_sign": ("float zf = q_min - rne(lo / s[p]);", "float zf = q_min + rne(lo / s[p]);"),
    "asym_range_not_widened_to_zero": ("float hi = 0.0f, lo = 0.0f;\n        for (int64_t r = 0; r < rows; r++)",
                                       "float hi = -INFINITY, lo = INFINITY;\n        for (int64_t r = 0; r < rows; r++)"),
    "asym_zero_point_subtracted_in_codes": ("c[m * ldc + k] = (int8_t)clampf(v + (float)z[p], q_min, q_max);",
                                            "c[m * ldc + k] = (int8_t)clampf(v - (float)z[p], q_min, q_max);"),
    "asym_weight_sum_term_added": ("v += t0 - t1 - t2 + t3;", "v += t0 + t1 - t2 + t3;"),
    "asym_constant_term_dropped": ("v += t0 - t1 - t2 + t3;", "v += t0 - t1 - t2;"),
    "asym_row_sum_term_dropped": ("v += t0 - t1 - t2 + t3;", "v += t0 - t1 + t3;"),
    "asym_fold_added": ("v -= (double)s_x[p] * (double)s_w[p * Q + q] * (double)z_x[p]", "v += (double)s_x[p] * (double)s_w[p * Q + q] * (double)z_x[p]"),
    "asym_fold_scale_index_transposed": ("v -= (double)s_x[p] * (double)s_w[p * Q + q] * (double)z_x[p]", "v -= (double)s_x[p] * (double)s_w[q * P + p] * (double)z_x[p]"),
    "segment_sum_skips_first": ("for (int64_t k = kb[p]; k < kb[p + 1]; k++) t += A[r * lda + k];",
                                "for (int64_t k = kb[p] + 1; k < kb[p + 1]; k++) t += A[r * lda + k];"),
    "silu_exponent_sign": ("return h / (1.0 + exp(-h));", "return h / (1.0 + exp(h));"),
    "gelu_half_dropped": ("return 0.5 * h * erfc(-h / sqrt(2.0));", "return h * erfc(-h / sqrt(2.0));"),
    "gelu_tanh_like_argument": ("return 0.5 * h * erfc(-h / sqrt(2.0));", "return 0.5 * h * erfc(-h / 2.0);"),
    "activation_rounded_twice": ("uint32_t bits = (uint32_t)sqo_bf16_from_f64(a) << 16;", "uint32_t bits = (uint32_t)sqo_bf16_from_f64((double)(float)a + 1e-3 * a) << 16;"),
    "geglu_halves_swapped": ("sqo_geglu((double)H[m * ld + k], (double)H[m * ld + K + k]);", "sqo_geglu((double)H[m * ld + K + k], (double)H[m * ld + k]);"),
    "geglu_gate_through_silu": ("return value * sqo_gelu(gate);", "return value * sqo_silu(gate);"),
    "geglu_gate_rounded_first": ("return value * sqo_gelu(gate);", "return value * (double)(float)sqo_gelu(gate) * (1.0 + 1e-3);"),
    "smooth_indexed_by_row": ("out[m * ldo + k] = X[m * ld + k] * mult[k];", "out[m * ldo + k] = X[m * ld + k] * mult[m % K];"),
    "per_row_uses_first_rows_scales": ("sqo_quantize_act_i8(X + m * ld, 1, K, ld, P, kb, s_pos + m * P,", "sqo_quantize_act_i8(X + m * ld, 1, K, ld, P, kb, s_pos,"),
    "per_row_scales_from_whole_matrix": ("sqo_calib_act(X + m * ld, 1, K, ld, P, kb, dual,", "sqo_calib_act(X, M, K, ld, P, kb, dual,"),
    "w4_nibbles_swapped": ("out[n * ldo + j] = (uint8_t)((Wq[n * ld + 2 * j] & 0xF) | ((Wq[n * ld + 2 * j + 1] & 0xF) << 4));",
                           "out[n * ldo + j] = (uint8_t)((Wq[n * ld + 2 * j + 1] & 0xF) | ((Wq[n * ld + 2 * j] & 0xF) << 4));"),
    "w4_unpack_without_sign": ("Wq[n * ld + 2 * j] = (int8_t)(((b & 0xF) ^ 8) - 8);", "Wq[n * ld + 2 * j] = (int8_t)(b & 0xF);"),
    "per_token_weight_scale_index_transposed": ("double sw = (double)s_w[n * P + p];", "double sw = (double)s_w[p * N + n];"),
    "per_token_act_scale_of_wrong_token": ("double t = (double)s_pos[m * P + p] * sw * acc_pos[i];", "double t = (double)s_pos[p] * sw * acc_pos[i];"),
    "per_token_negative_path_uses_positive_scale": ("double u = (double)s_neg[m * P + p] * sw * acc_neg[i];", "double u = (double)s_pos[m * P + p] * sw * acc_neg[i];"),
    "bf16_truncates": ("double q = nearbyint((f * 2.0 - 1.0) * 128.0);", "double q = floor((f * 2.0 - 1.0) * 128.0);"),
}


def _run_mutation(name, workdir):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    if src.count(old) < 1:
        return None, f"mutation anchor for {name} no longer in the oracle source"
    mutated = os.path.join(workdir, name + ".c")
    with open(mutated, "w") as f:
        f.write(src.replace(old, new))
    lib = os.path.join(workdir, "lib" + name + ".so")
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", lib, mutated, "-lm"])
    env = dict(os.environ, SEGQUANT_ORACLE_LIB=lib, OMP_NUM_THREADS="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       env=env, cwd=ROOT, capture_output=True, text=True)
    return r.returncode, r.stdout[-2000:]


@pytest.fixture(scope="module")
def mutation_results(tmp_path_factory):
    """All mutated builds run the pin suite side by side (they are independent processes)."""
    from concurrent.futures import ThreadPoolExecutor
    workdir = str(tmp_path_factory.mktemp("mutants"))
    names = sorted(MUTATIONS)
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        return dict(zip(names, pool.map(lambda n: _run_mutation(n, workdir), names)))


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_reject_planted_mistake(name, mutation_results):
    rc, tail = mutation_results[name]
    assert rc is not None, tail
    assert rc == 1, f"pins did not catch '{name}':\n{tail}"
