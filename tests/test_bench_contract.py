"""The benchmark's reference arm runs without a GPU: its one JSON line carries the keys the contract names."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference"
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in d, key
    assert d["config"]["workload"] == "tiny" and "model" not in d["config"]
    assert d["vs_baseline"] is None and d["higher_is_better"] is True and d["data"] == "synthetic"
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == d["value"]
    e2e = d["e2e"]
    assert e2e["value"] == d["value"] and e2e["unit"] == d["unit"]
    assert e2e["h2d_bytes_per_step"] == 0 and e2e["d2h_bytes_per_step"] == 0
    assert d["gpu_launches"] == 0 and d["value"] > 0
    # the arm honours --steps / --warmup and validates its row sampling where the oracle can run every row
    assert d["steps"] == 1 and d["warmup"] == 0
    chk = cb["sampling_check"]
    assert chk["workload"] == "single_view" and 0.7 <= chk["ratio"] <= 1.4
    for key in ("workload", "batch_per_gpu", "seq_len", "packed_len", "heads", "head_dim", "keep", "k_core", "k_anchor",
                "refresh_interval", "step", "tokens_per_step", "l2", "parallelism", "timing", "stage_timing"):
        assert key in d["config"], key


import pytest


@pytest.mark.gpu
def test_gpu_arm_prints_one_contract_line():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "single_view", "--steps", "3",
                          "--warmup", "3", "--cpu-seconds", "1", "--also", "tiny"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] >= 3 and d["dtype"] == "bf16"
    roof = d["roofline"]
    for key in ("bound", "achieved", "peak", "unit", "frac", "traffic"):
        assert key in roof, key
    assert roof["bound"] in ("hbm", "tensor", "alu") and abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-3
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] > 0
    e2e = d["e2e"]
    assert e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0 and 0 < e2e["value"] < d["value"]
    assert d["gpu_launches"] > 0 and d["value"] > 0
    assert "sm_mhz" in d["clocks"] and "reasons" in d["clocks"]
    # two regimes, each with its own clock record; the steady one is the headline
    assert d["value_burst"] > 0 and d["ms_per_step_burst"] > 0 and "sm_mhz" in d["clocks_burst"]
    assert d["clocks"]["replays_before_timed_region"] * d["ms_per_step"] >= 900      # >= 1 s of run-in (minus noise)
    assert abs(roof["burst"]["frac"] - roof["burst"]["achieved"] / roof["burst"]["peak"]) < 1e-3
    assert roof["exp2"]["bound"] == "exp2" and roof["exp2"]["peak"] > 0
    # selection is reported against the launch floor, not against memory bandwidth
    sel = d["stages"]["select"]
    assert sel["bound"] == "latency" and 0 < sel["launch_floor_us"] < sel["us"]
    # the steps sum to the cycle they are quoted beside (same regime), within timing noise
    assert d["full_step_us"] + d["sparse_step_us"] <= 1.15 * d["ms_per_step"] * 1e3
    # the other shapes ride along with the same keys
    also = d["also"]["tiny"]
    for key in ("value", "value_burst", "ms_per_step", "clocks", "roofline", "stages", "e2e", "config"):
        assert key in also, key
    assert also["config"]["workload"] == "tiny"
    assert sorted(also["config"]) == sorted(d["config"])
