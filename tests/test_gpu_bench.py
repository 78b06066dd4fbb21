"""bench.py on a GPU: one JSON line with the agreed keys, on a small configuration."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), *flags]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


@pytest.mark.parametrize("config,variant", [("2", "carry"), ("2", "two_pass"), ("4", "carry")])
def test_bench_line_has_the_agreed_keys(config, variant):
    flags = ["--config", config, "--variant", variant, "--steps", "6", "--warmup", "3", "--e2e-steps", "2",
             "--cpu-steps", "1"]
    if config == "4":
        flags += ["--max-elements", "400000"]        # a prefix of the ResNet-18 tensors: seconds, not minutes
    line = _run(*flags)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
                "roofline", "cpu_baseline"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 6 and line["warmup"] == 3
    assert line["unit"] == "GB/s" and line["value"] > 0 and line["ms_per_step"] > 0
    assert line["higher_is_better"] is True and line["scaling"] == "weak" and line["vs_baseline"] is None
    assert line["data"] == "synthetic" and "workload" in line["config"]
    assert line["config"]["variant"] == variant
    assert line["config"]["bytes_per_element_step"] == (16 if variant == "carry" else 24)
    assert line["gpu_launches"] >= 6                                   # at least one kernel per step
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == 2 * e2e["d2h_bytes_per_step"] > 0
    roof = line["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 0
    assert roof["frac"] is None or abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    # the captured DRAM traffic, or null together with the reason
    assert "traffic" in roof and roof["traffic_sources_hash"]
    assert roof["traffic"] is not None or "traffic_stale_since" in roof or "traffic_note" in roof
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and cpu["sample"]
    assert set(line["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    for bad in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"):
        assert bad not in line["clocks"]["reasons"]
