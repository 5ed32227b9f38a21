"""bench.py prints one JSON line with the keys its contract names (a short run on the small workload)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, out.stdout[-2000:]                       # stdout carries the one JSON line only
    return json.loads(lines[0])


def test_main_line_has_the_contract_keys():
    d = run_bench("--workload", "cfg3", "--steps", "20", "--warmup", "3", "--no-all")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "roofline", "e2e", "cpu_baseline", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 20 and d["warmup"] >= 3 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic"
    r = d["roofline"]
    trains = r["trains_ms_per_step"]
    assert d["config"]["workload"] == "cfg3" and d["gpu_launches"] == 20 * trains["n_trains"] and trains["n_trains"] >= 3
    assert trains["min"] <= trains["median"] <= trains["max"] and abs(trains["median"] - d["ms_per_step"]) < 1e-6
    assert len(d["config"]["input_checksum"]) == 16 and list(d["per_config"]) == ["cfg3"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3 and r["traffic"] > 0
    assert abs(d["value"] - r["achieved"]) < 1e-6 and d["value"] > 1000
    # beside the train of launches: the library's own copy over the same buffers, and launches timed one by one
    assert r["own_copy"]["GB/s"] > 1000 and 0.5 < r["own_copy"]["softmax_over_copy_time"] < 2.0
    assert r["single_launch_ms"]["best"] <= r["single_launch_ms"]["median"] and r["single_launch_ms"]["n"] == 20
    assert 0.9 < r["traffic_over_algorithmic"] < 1.3                 # eight consecutive launches: the write-back is counted
    e = d["e2e"]
    assert e["value"] > 1 and e["h2d_bytes_per_step"] == e["d2h_bytes_per_step"] == 131072 * 128 * 2
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and "sample" in c
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])


def test_reference_arm_line():
    d = run_bench("--impl", "reference", "--workload", "cfg1", "--steps", "2", "--warmup", "1")
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
