"""The one JSON line bench.py prints: its keys and types, for the oracle arm (CPU) and for the CUDA arm (-m gpu), on a
workload cut down to a few requests so that either run takes seconds."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SMALL = ["--requests", "2", "--layers", "2", "--context", "3000", "--steps", "2", "--warmup", "3"]


def run_bench(extra):
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + SMALL + extra, cwd=ROOT, capture_output=True,
                       text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, "bench.py must print exactly one line"
    return json.loads(lines[0])


def check_common(j):
    assert j["metric"] == "resolved selections/s" and j["unit"] == "selections/s"
    assert j["n_gpus"] == 1 and j["steps"] == 2 and j["warmup"] == 3
    assert j["higher_is_better"] is True and j["scaling"] == "weak" and j["vs_baseline"] is None
    assert j["data"] == "synthetic" and j["dtype"] == "int32/u8"
    assert j["config"]["workload"] == "c2_dsa_decode" and "model" not in j["config"]
    assert j["value"] > 0 and j["ms_per_step"] > 0
    for key in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert key in j["e2e"]


def test_reference_arm_line():
    j = run_bench(["--impl", "reference"])
    check_common(j)
    assert j["impl"] == "reference"
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == j["value"] and cb["sample"]
    assert j["e2e"]["value"] == j["value"] and j["e2e"]["h2d_bytes_per_step"] == 0 and j["e2e"]["d2h_bytes_per_step"] == 0


@pytest.mark.gpu
def test_cuda_arm_line():
    j = run_bench(["--no-per-config", "--cpu-sample-steps", "5"])
    check_common(j)
    assert "impl" not in j or j["impl"] != "reference"
    assert j["gpu_launches"] > 0 and j["status_bits"] == 0
    assert j["e2e"]["value"] > 0 and j["e2e"]["h2d_bytes_per_step"] > 0 and j["e2e"]["d2h_bytes_per_step"] > 0
    c = j["clocks"]
    assert c["sm_max_mhz"] >= c["sm_mhz"] > 0 and isinstance(c["reasons"], list)
    r = j["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in r
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    a = j["roofline_all_hit"]
    assert a["bound"] == "hbm" and abs(a["frac"] - a["achieved"] / a["peak"]) < 1e-9 and a["traffic"] > 0
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1 and cb["sample"]
