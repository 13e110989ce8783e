"""bench.py run for real on a small workload: the JSON line carries what the
measurement contract asks for, and the side modes print their own lines."""
from __future__ import annotations

import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    return json.loads(out.stdout.strip().splitlines()[-1])


def test_bench_line_of_a_small_workload_has_every_contract_key():
    line = _run("--workload", "tiny_ragged", "--steps", "5", "--warmup", "3")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config",
                "roofline", "cpu_baseline", "e2e", "clocks", "gpu_launches"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 5 and line["value"] > 0
    assert line["config"]["workload"] == "tiny_ragged" and "model" not in line["config"]
    assert line["gpu_launches"] > 0
    r = line["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    e = line["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < line["value"]                  # the link, not HBM, bounds the host-fed path
    c = line["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1
    assert line["clocks"]["sm_max_mhz"] >= line["clocks"]["sm_mhz"] > 0


def test_scan_and_pack_modes_print_their_lines():
    scan = _run("--scan", "--workload", "tiny_ragged", "--steps", "5")
    assert scan["workload"] == "tiny_ragged" and scan["scan"]["gbs_median"] > 0
    assert scan["norm"] > 0
    pack = _run("--pack", "--workload", "tiny_ragged", "--steps", "5")
    assert len(pack["pack"]) == 2
    for row in pack["pack"]:
        assert row["pack"]["gbs"] > 0 and row["unpack"]["gbs"] > 0
