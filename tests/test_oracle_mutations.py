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
