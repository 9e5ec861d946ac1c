"""The benchmark's JSON line on the smallest workload: every key of the contract is present and
consistent (one GPU; the figures themselves are not judged here)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_json_line_of_the_smallest_workload():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "cfg1", "--steps", "4", "--warmup", "3",
                        "--no-per-config"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["n_gpus"] == 1 and j["warmup"] == 3 and j["steps"] >= 4
    assert j["higher_is_better"] is True and j["scaling"] == "weak" and j["vs_baseline"] is None
    assert j["data"] == "synthetic" and j["config"]["workload"] == "cfg1"
    assert j["value"] > 0 and j["ms_per_step"] > 0 and j["unit"] == "TFLOP/s"
    assert j["gpu_launches"] == 2 * j["steps"] * len(j["config"]["shapes_MKN"])    # rotate+quantize and GEMM per layer
    assert set(j["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    e = j["e2e"]
    assert e["value"] > 0 and e["unit"] == j["unit"]
    M, K, N = j["config"]["shapes_MKN"][0]
    assert e["h2d_bytes_per_step"] == 2 * M * K and e["d2h_bytes_per_step"] == 2 * M * N
    roof = j["roofline"]
    assert roof["bound"] == "tensor" and roof["unit"] == "TFLOP/s"
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert "traffic" in roof and roof["traffic"] is None        # no ncu capture is recorded for this workload
    eff = roof["operand_data_effect"]
    assert eff["MKN"] == [M, K, N] and eff["us_real_operands"] > 0 and eff["us_zero_codes"] > 0
    cpu = j["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["cores"] >= 1 and cpu["sample"]
    assert j.get("notes") is None
