"""bench.py prints one JSON line with the agreed keys: the reference arm (CPU oracle) here, the CUDA arm on a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"}


def _last_json_line(text):
    lines = [ln for ln in text.splitlines() if ln.startswith("{")]
    assert lines, text[-2000:]
    return json.loads(lines[-1])


def test_reference_arm_line():
    r = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--config", "0", "--steps", "2", "--warmup", "1"],
                       cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    j = _last_json_line(r.stdout)
    assert BASE_KEYS <= set(j) and j["impl"] == "reference"
    assert j["unit"] == "GB/s" and j["value"] > 0 and j["higher_is_better"] is True and j["vs_baseline"] is None
    assert j["config"]["workload"] == "tiny-100k" and j["data"] == "synthetic"
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == 1 and cb["value"] == j["value"] and "sample" in cb
    assert j["e2e"] == {"value": j["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert j["gpu_launches"] == 0


@pytest.mark.gpu
def test_cuda_arm_line():
    r = subprocess.run([sys.executable, "bench.py", "--config", "1", "--steps", "5", "--warmup", "3", "--no-cpu-baseline"],
                       cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    j = _last_json_line(r.stdout)
    assert BASE_KEYS | {"roofline", "clocks", "kernels"} <= set(j) and "impl" not in j
    assert j["n_gpus"] == 1 and j["steps"] == 5 and j["warmup"] == 3 and j["scaling"] == "weak"
    assert j["config"]["workload"] == "resnet18-11.2M" and j["dtype"] == "f32"
    rf = j["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and rf["peak"] > 1000
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9 and 0.05 < rf["frac"] < 1.3
    assert j["gpu_launches"] == 4 * 5                       # statistics (2 launches), compress, aggregate per step
    e = j["e2e"]
    assert 0 < e["value"] < j["value"] and e["h2d_bytes_per_step"] >= 8 * 11_200_000 * 4 and e["d2h_bytes_per_step"] >= 4 * 11_200_000
    assert j["clocks"]["sm_mhz"] > 0 and isinstance(j["clocks"]["reasons"], list)
