"""bench.py prints one JSON line with the keys its callers rely on: the CPU-oracle arm on the
small workload here, the GPU arm on a B200."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline"}


def run_bench(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                       cwd=ROOT, timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [x for x in r.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line():
    line = run_bench("--impl", "reference", "--config", "0", "--steps", "1", "--warmup", "0")
    assert BASE_KEYS <= set(line)
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["metric"] == "FO-SGD round-trip gradient elems/s" and line["unit"] == "elems/s"
    assert line["value"] > 0 and line["e2e"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("cfg0")


@pytest.mark.gpu
def test_gpu_arm_line():
    line = run_bench("--config", "1", "--steps", "5", "--warmup", "3")
    assert BASE_KEYS | {"clocks", "gpu_launches", "roofline", "path_roofline", "paths", "kernels"} <= set(line)
    assert "impl" not in line and line["n_gpus"] == 1 and line["steps"] == 5 and line["warmup"] == 3
    assert line["value"] > 0 and line["gpu_launches"] >= 5 * 8
    r = line["roofline"]
    assert {"bound", "achieved", "peak", "unit", "frac", "traffic"} <= set(r)
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    # the fraction is on the method's own bytes; the kernel's own traffic (intermediates included) is listed apart
    assert r["algorithmic_bytes_per_launch"] <= r["implementation_bytes_per_launch"]
    assert r["frac"] <= r["implementation_frac"] + 1e-12 and r["call"]["frac"] <= r["implementation_frac"]
    assert set(r["per_kernel"]) == set(line["kernels"])
    assert line["repeats"] >= 1 and line["clocks"]["samples"] >= 10
    assert line["path_roofline"]["alu_peak_source"].startswith("measured") and line["alu_probe"]["lane_ops_per_s"]["fadd"] > 1e13
    e = line["e2e"]
    assert e["h2d_bytes_per_step"] == 16 * (1 << 20) * 4 and e["d2h_bytes_per_step"] == (1 << 20) * 4
    assert 0 < e["value"] < line["value"]
    c = line["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    assert line["config"]["workload"].startswith("cfg1") and "l2" in line["config"]
    assert set(line["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
