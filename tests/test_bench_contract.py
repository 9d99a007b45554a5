"""The JSON lines bench.py prints: required keys and their shapes, for the reference arm (CPU only) and for
the library's own arm (needs a GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
             "dtype", "data", "config", "e2e", "cpu_baseline"}


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, cwd=ROOT, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line():
    d = _run("--impl", "reference", "--config", "tiny_fl_fsdp", "--steps", "1", "--warmup", "1")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["metric"] == "synced_params_per_s" and d["unit"] == "params/s" and d["higher_is_better"] is True
    assert d["vs_baseline"] is None and d["data"] == "synthetic" and d["config"]["workload"] == "tiny_fl_fsdp"
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == cb["host_cores"] >= 1 and cb["value"] == d["value"]
    assert cb["one_core"]["cores"] == 1 and cb["one_core"]["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["value"] > 0


@pytest.mark.gpu
def test_own_arm_line():
    d = _run("--config", "tiny_fl_fsdp", "--steps", "8", "--warmup", "3")
    assert BASE_KEYS <= set(d) and "impl" not in d
    assert d["metric"] == "synced_params_per_s" and d["n_gpus"] == 1 and d["steps"] == 8 and d["warmup"] == 3
    assert d["scaling"] == "weak" and d["dtype"] == "f32" and d["config"]["workload"] == "tiny_fl_fsdp"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    assert d["gpu_launches"] > 0 and set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] == 2 * 4 * 1_000_032 * 2 and e["d2h_bytes_per_step"] == 8
    assert e["value"] < d["value"]                       # copies inside the timed region can only slow it down
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    assert c["one_core"]["cores"] == 1 and c["one_core"]["value"] > 0
    assert "other_workloads" not in d                    # only the default workload brings the other two along
    # value = G * P * steps / time
    assert abs(d["value"] - 2 * 1_000_003 * 8 / (d["ms_per_step"] * 8 / 1e3)) / d["value"] < 1e-6
