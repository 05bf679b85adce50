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


def test_traffic_table_names_workloads_and_goes_stale_with_the_kernel_source():
    assert set(bench.GEMM_DRAM_TRAFFIC) <= set(WL.WORKLOADS)
    for e in bench.GEMM_DRAM_TRAFFIC.values():
        assert isinstance(e["bytes"], int) and e["bytes"] > 0 and len(e["source_tag"]) == 16 and e["from"]
    assert bench.gemm_dram_traffic("no_such_workload")[0] is None
    saved = dict(bench.GEMM_DRAM_TRAFFIC)
    try:
        bench.GEMM_DRAM_TRAFFIC["tiny_qkv"] = {"bytes": 123, "source_tag": "0" * 16, "from": "test"}
        assert bench.gemm_dram_traffic("tiny_qkv")[0] is None                      # another kernel source: stale
        bench.GEMM_DRAM_TRAFFIC["tiny_qkv"]["source_tag"] = bench.gemm_source_tag()
        assert bench.gemm_dram_traffic("tiny_qkv") == (123, "test")
    finally:
        bench.GEMM_DRAM_TRAFFIC.clear()
        bench.GEMM_DRAM_TRAFFIC.update(saved)


def test_fractions_against_the_three_peaks():
    p8 = bench.eight_bit_peaks({"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0})
    assert p8 == {"burst": 3200.0, "sustained": 2800.0, "nominal": 4500.0}
    f = bench.fractions(1600.0, p8)
    assert f == {"of_measured_burst": 0.5, "of_measured_sustained": round(1600 / 2800, 4), "of_nominal_4500": round(1600 / 4500, 4)}


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
