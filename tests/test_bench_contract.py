"""bench.py's reference arm (the CPU oracle) prints one JSON line with the contract's keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1",
                          "--ref-budget-s", "3"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["steps"] == 2 and d["warmup"] == 1 and d["vs_baseline"] is None
    assert d["unit"] == "TOPS" and d["value"] > 0 and d["higher_is_better"] is True and d["data"] == "synthetic"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert "workload" in d["config"]


def test_non_zero_ranks_of_the_reference_arm_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


import pytest


@pytest.mark.gpu
def test_gpu_arm_prints_the_contract_line_with_roofline_and_e2e():
    """The library's own arm on one GPU: one JSON line with the contract's keys, a roofline object
    for the dominant call, an end-to-end figure with its copy sizes, and a non-zero launch count."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "14", "--warmup", "3", "--no-cpu-baseline",
                          "--no-legs"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "e2e", "gpu_launches", "roofline", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 14 and d["unit"] == "TOPS" and d["value"] > 0 and d["vs_baseline"] is None
    assert d["gpu_launches"] == 14 * 3 and d["device_status"] == 0 and d["e2e"]["device_status"] == 0
    r = d["roofline"]
    assert r["bound"] in ("hbm", "tensor", "alu") and 0 < r["frac"] < 1.5 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert len(r["calls"]) == 3 and abs(sum(c["share"] for c in r["calls"]) - 1.0) < 1e-9
    # the calls timed one by one add up to the step (they overlap a little inside it)
    assert 0.8 < d["sum_call_ms_per_step"] / d["sustained"]["ms_per_step"] < 1.25
    assert d["sustained"]["seconds"] >= 0.5 and d["clocks"]["samples"] >= 4
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 4 * 12800 * 512 and e["d2h_bytes_per_step"] == 4 * 12800 * 512 and 0 < e["value"] < d["value"]
    assert "workload" in d["config"] and "model" not in d["config"]
