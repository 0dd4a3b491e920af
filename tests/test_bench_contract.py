"""The benchmark's output contract: the LAST stdout line is one compact JSON object with the agreed keys.

A line that is too long to survive in a truncated log tail, or that lacks `value`, `roofline`,
`cpu_baseline` or `e2e`, makes a whole run unreadable for whoever collects it, so both arms are run here as
subprocesses and their last lines are parsed."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline"}


def last_line(args, timeout):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True, text=True,
                         timeout=timeout, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    return lines, json.loads(lines[-1])


def test_reference_arm_prints_the_oracle_line():
    lines, obj = last_line(["--impl", "reference", "--steps", "20", "--warmup", "5"], 120)
    assert len(lines) == 1
    assert BASE_KEYS <= set(obj) and obj["impl"] == "reference"
    assert obj["value"] > 0 and obj["unit"] == "us" and obj["higher_is_better"] is False
    assert obj["steps"] == 20 and obj["warmup"] == 5 and obj["vs_baseline"] is None
    assert obj["config"]["workload"] == "ar_n8_512KiB"
    cb = obj["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] == obj["value"] and cb["cores"] >= 1 and cb["sample"]
    assert obj["e2e"] == {"value": obj["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_gpu_arm_last_line_is_compact_and_complete():
    lines, obj = last_line(["--quick", "--steps", "20", "--warmup", "5"], 600)
    assert len(lines[-1]) < 2000                                   # survives in a truncated tail
    assert BASE_KEYS | {"roofline", "clocks", "gpu_launches", "replays"} <= set(obj)
    assert obj["metric"] == "allreduce_latency_us" and obj["unit"] == "us" and 0.5 < obj["value"] < 50.0
    assert obj["steps"] == 20 and obj["warmup"] >= 3 and obj["n_gpus"] == 1
    assert abs(obj["ms_per_step"] * 1e3 - obj["value"]) < 1e-3
    roof = obj["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 1000
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-3 and 0.05 < roof["frac"] < 1.2
    assert roof["traffic"] is None or roof["traffic"] > 0
    assert obj["gpu_launches"] == obj["steps"] * obj["replays"] * max(1, 1000 // obj["steps"])
    e2e = obj["e2e"]
    assert e2e["value"] > obj["value"] and e2e["h2d_bytes_per_step"] == 8 * 524288 == e2e["d2h_bytes_per_step"]
    assert obj["cpu_baseline"]["kind"] == "oracle" and obj["cpu_baseline"]["value"] > 0
    assert obj["config"]["workload"] == "ar_n8_512KiB" and "model" not in obj["config"]
    assert obj["device_status"] == 0
    # every earlier line is a detail section of its own
    for ln in lines[:-1]:
        d = json.loads(ln)
        assert set(d) == {"detail", "data"}
