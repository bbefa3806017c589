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
    r = subprocess.run([sys.executable, "bench.py", "--config", "1", "--steps", "5", "--warmup", "3", "--no-cpu-baseline",
                        "--no-workloads"], cwd=ROOT, capture_output=True, text=True, timeout=900)
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
    assert j["workloads"] is None
    for name in ("tq_compress", "tq_decompress_aggregate"):
        k = j["kernels"][name]
        assert 0 < k["ms_min"] <= k["ms_median"] and k["ms_min"] <= k["ms"]
        assert abs(k["frac_of_hbm_peak"] - k["algorithmic_bytes"] / (k["ms"] * 1e-3) / 1e9 / rf["peak"]) < 1e-9


@pytest.mark.gpu
def test_cuda_arm_line_carries_every_large_workload():
    """The default line (headline: 25.6 M x 16) also reports, per kernel, the bf16 workload (uniform and non-uniform,
    4 and 16 levels) and the 10^9-element workload: time as median / min / mean, algorithmic bytes, fraction of the
    copy peak, and the clocks sampled while that workload ran."""
    r = subprocess.run([sys.executable, "bench.py", "--steps", "5", "--warmup", "3", "--no-cpu-baseline", "--no-e2e"],
                       cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stderr[-2000:]
    j = _last_json_line(r.stdout)
    assert j["config"]["workload"] == "resnet50-25.6M"
    wl = j["workloads"]
    want = {f"gpt2s-124M-bf16-g3.0-{m}-L{L}" for m in ("uniform", "nonuniform") for L in (4, 16)} | {"flat-1e9"}
    assert set(wl) == want
    peak = j["roofline"]["peak"]
    for name, r2 in wl.items():
        assert r2["ms_per_step"] > 0 and r2["clocks"]["sm_mhz"] > 0 and isinstance(r2["clocks"]["reasons"], list)
        for kn in ("tq_compress", "tq_decompress_aggregate"):
            k = r2["kernels"][kn]
            assert 0 < k["ms_min"] <= k["ms_median"]
            assert abs(k["frac_of_hbm_peak"] - k["algorithmic_bytes"] / (k["ms"] * 1e-3) / 1e9 / peak) < 1e-9
            assert 0.05 < k["frac_of_hbm_peak"] < 1.3
    n, d = 8, 124_000_000
    assert wl["gpt2s-124M-bf16-g3.0-uniform-L16"]["kernels"]["tq_compress"]["algorithmic_bytes"] == n * d * 2 + n * d * 4 // 8
    assert wl["flat-1e9"]["kernels"]["tq_decompress_aggregate"]["algorithmic_bytes"] == 4 * 10**9 * 3 // 8 + 4 * 10**9
