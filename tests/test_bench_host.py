"""Host-side arithmetic of bench.py (no GPU): op and byte counts per layer, the traffic table's keys, and the
shape of the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import bench
from paper_2507_14811_b200 import workloads as WL

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_op_and_byte_counts():
    adaln, fc2 = WL.WORKLOADS["dit_xl2"]
    executed, useful = bench.layer_ops(adaln)
    assert useful == 2 * 2048 * 6912 * 1152 and executed == 2 * useful          # dual: two GEMMs
    fc1 = WL.WORKLOADS["sd3_mmdit"][1]
    assert bench.layer_ops(fc1) == (2.0 * 8858 * 6144 * 1536, 2.0 * 8858 * 6144 * 1536)
    # GEMM: both code matrices + weight codes + bf16 output; quantize: bf16 in + one byte per code matrix
    assert bench.gemm_bytes(fc2) == 2048 * 4608 * 2 + 1152 * 4608 + 2 * 2048 * 1152
    assert bench.quant_bytes(fc2) == 2048 * 4608 * (2 + 2)
    assert bench.quant_bytes(fc1) == 8858 * 1536 * (2 + 1)
    assert bench.layer_ops(fc2, M=100)[1] == 2.0 * 100 * 1152 * 4608


def test_traffic_table_names_workloads():
    assert set(bench.GEMM_DRAM_TRAFFIC) <= set(WL.WORKLOADS)
    assert all(isinstance(v, int) and v > 0 for v in bench.GEMM_DRAM_TRAFFIC.values())


def test_measured_peaks_have_the_fields_the_roofline_uses():
    p = bench.measured_peaks()
    assert p["hbm_gbs"] > 1000 and p["bf16_tflops"] > 100 and p["source"] in ("measured", "fallback")


def test_reference_arm_prints_one_json_line_on_the_tiny_workload():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_qkv",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TOPS" and d["value"] > 0 and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["config"]["workload"] == "tiny_qkv"
