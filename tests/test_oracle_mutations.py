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
    "bf16_truncates": ("double q = nearbyint((f * 2.0 - 1.0) * 128.0);", "double q = floor((f * 2.0 - 1.0) * 128.0);"),
}


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_pins_reject_planted_mistake(name, tmp_path):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation anchor for {name} no longer in the oracle source"
    mutated = tmp_path / "mutated.c"
    mutated.write_text(src.replace(old, new))
    lib = tmp_path / "libmutated.so"
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", str(lib), str(mutated), "-lm"])
    env = dict(os.environ, SEGQUANT_ORACLE_LIB=str(lib))
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       env=env, cwd=ROOT, capture_output=True, text=True)
    assert r.returncode == 1, f"pins did not catch '{name}':\n{r.stdout[-2000:]}"
