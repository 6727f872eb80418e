"""The benchmark's output contract, on the tiny workload (seconds): one JSON line with the keys the
driver reads, device-timed values, launch counts, the roofline and CPU-baseline objects."""
import json
import os
import subprocess
import sys

import pytest

from gpu_common import engine, requires_gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@requires_gpu
def test_bench_prints_one_json_line_with_the_contract_keys():
    engine()
    r = subprocess.run([sys.executable, "bench.py", "--workload", "cfg1_tiny", "--steps", "2", "--warmup", "3"],
                       cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, r.stdout[-2000:]
    j = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in j, key
    assert j["n_gpus"] == 1 and j["steps"] == 2 and j["warmup"] == 3
    assert j["value"] > 0 and j["ms_per_step"] > 0 and j["higher_is_better"] is True
    assert j["scaling"] == "weak" and j["data"] == "synthetic" and j["dtype"] == "bf16" and j["vs_baseline"] is None
    assert j["config"]["workload"] == "cfg1_tiny" and "model" not in j["config"]
    assert j["gpu_launches"] > 0
    e = j["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] != j["value"]                       # measured separately, host copies inside the timed region
    ro = j["roofline"]
    assert ro["bound"] == "hbm" and ro["unit"] == "GB/s" and ro["peak"] > 0 and ro["achieved"] > 0
    assert abs(ro["frac"] - ro["achieved"] / ro["peak"]) < 1e-9
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1 and cb["sample"]
    assert set(j["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
