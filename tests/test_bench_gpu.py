"""bench.py on the GPU, small workload: the one JSON line carries every field of the measurement contract."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_fields():
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "n512", "--steps", "200",
                                   "--warmup", "3", "--no-autotune", "--no-per-config"], cwd=ROOT, text=True, timeout=900)
    line = json.loads(out.strip().splitlines()[-1])          # the last line of stdout
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline", "per_config"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 200 and line["dtype"] == "f64" and line["data"] == "synthetic"
    assert line["higher_is_better"] is True and line["vs_baseline"] is None and line["unit"] == "GFLOP/s"
    assert line["config"]["workload"].startswith("n512") and "model" not in line["config"]
    assert line["value"] == pytest.approx(2 * 512 ** 3 / (line["ms_per_step"] * 1e-3) / 1e9)
    assert line["gpu_launches"] == 200 * 1                   # one fused launch per product
    r = line["roofline"]
    assert r["bound"] == "alu" and r["unit"] == "TFLOP/s" and 0 < r["frac"] <= 1.05 and r["frac"] == pytest.approx(r["achieved"] / r["peak"])
    e = line["e2e"]
    assert e["h2d_bytes_per_step"] == 2 * 512 * 512 * 8 and e["d2h_bytes_per_step"] == 512 * 512 * 8 and 0 < e["value"] < line["value"]
    c = line["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    assert c["max_err_on_sample"] <= line["parity"]["bound"] and line["parity"]["int_equal"] is True
    assert set(line["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    p = line["path_roofline"]
    assert 0 < p["frac"] <= 1.0 and 0 < p["frac_of_floor"] <= 1.0
