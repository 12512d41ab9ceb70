"""bench.py on the GPU at a reduced size: the one JSON line carries every key of the measurement contract, for the
default arm (one column shard per GPU) and for the one-process-per-parameter-server arm."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-3000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


def _common(line, steps, warmup):
    assert line["unit"] == "GB/s" and line["metric"].startswith("N-of-(N+b) aggregate+update")
    assert line["n_gpus"] == 1 and line["steps"] == steps and line["warmup"] == warmup
    assert line["value"] > 0 and line["ms_per_step"] > 0 and line["higher_is_better"] is True
    assert line["vs_baseline"] is None and line["data"] == "synthetic" and line["dtype"] == "f32"
    assert line["config"]["workload"].startswith("c1_") and "model" not in line["config"]
    roof = line["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9 and "traffic" in roof
    assert line["gpu_launches"] == steps
    assert set(line["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_default_arm_prints_the_contract_line(cuda_device):
    line = _run("--columns", "400000", "--steps", "4", "--warmup", "3", "--only-headline", "--cpu-steps", "1")
    _common(line, 4, 3)
    assert line["scaling"] == "weak"
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["unit"] == "GB/s"
    assert e2e["h2d_bytes_per_step"] == 96 * 400000 * 4 + 100 * 8 and e2e["d2h_bytes_per_step"] > 400000 * 4
    cpu = line["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["value"] > 0 and cpu["unit"] == "GB/s" and cpu["cores"] >= 1 and cpu["sample"]
    assert cpu["single_thread"]["cores"] == 1
    assert line["extra"]["separate_calls_launches_per_step"] == 3
    # a reduced size is not the workload the ncu traffic figure was taken on
    assert line["roofline"]["traffic"] is None


def test_parameter_server_arm_prints_the_contract_line(cuda_device):
    line = _run("--servers", "--columns", "400000", "--steps", "4", "--warmup", "3")
    _common(line, 4, 3)
    assert line["scaling"] == "strong" and line["e2e"] is None and line["cpu_baseline"] is None
    assert "parameter servers" in line["config"]["sharding"] and line["roofline"]["link_bytes_per_step"] == 0
