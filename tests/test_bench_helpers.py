"""Host-side helpers of bench.py (no GPU): the DRAM-traffic table scales with the rows of a launch, the
argument parser knows every kernel family, and the reference arm's line has the contract's keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def test_traffic_table_scales_with_rows():
    rows, nbytes = bench.NCU_TRAFFIC[2]
    assert bench.ncu_traffic(2, rows) == nbytes
    assert bench.ncu_traffic(4, 32768) == 8 * bench.ncu_traffic(4, 4096)
    assert set(bench.NCU_TRAFFIC) == {1, 2, 3, 4, 5}


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "1", "--ref-rows", "256"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["value"] > 0 and line["higher_is_better"] is True
