"""bench.py on a GPU: one JSON line carrying every key of the measurement
contract, with values in a sane range."""
import json
import os
import subprocess
import sys

import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_every_contract_key():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3"],
                       capture_output=True, text=True, timeout=900)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, "rank 0 prints exactly one line"
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 5 and d["warmup"] >= 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["data"] == "synthetic" and d["config"]["workload"] == "qwen2304" and "model" not in d["config"]
    assert abs(d["value"] - d["config"]["algorithmic_bytes_per_step"] / (d["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * d["value"]
    assert 2000.0 < d["value"] < 9000.0, "a full prologue step must be HBM-bound on a B200"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["traffic"] is None or r["traffic"] > 0.5 * r["algorithmic_bytes_per_launch"]
    assert r["same_loop_torch_copy_of_the_same_bytes"]["us"] > 0.5 * r["us_per_launch"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and "sample" in c
    assert c["all_cores"]["cores"] == len(os.sched_getaffinity(0)) and c["all_cores"]["value"] > 0
    par = c["parity_on_sample"]
    assert par["v_bit_exact"] is True
    for t in ("q", "k"):
        assert par[t]["n_beyond_tolerance"] == 0 and par[t]["n"] > 1e6 and sum(par[t]["ulp_hist"].values()) == par[t]["n"]
    rep = d["repeats"]
    assert rep["n"] == 5 and rep["steps_each"] * rep["us_per_layer_median"] >= 19e3
    assert rep["us_per_layer_min"] <= rep["us_per_layer_median"] <= rep["us_per_layer_max"]
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == e["d2h_bytes_per_step"] == d["config"]["algorithmic_bytes_per_step"] // 2
    assert 0 < e["value"] < d["value"]
    assert d["gpu_launches"] == 2 * d["steps"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    for bad in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"):
        assert bad not in d["clocks"]["reasons"]
    pc = d["per_config"]
    assert set(pc) >= {"launch_floor", "tiny", "sd3", "qwen768", "temporal", "temporal_steps", "next_rows_temporal"}
    ts = pc["temporal_steps"]
    sel = ts["steps_1_to_7_selective"]
    assert [row["step"] for row in sel["per_step"]] == list(range(1, 8))
    assert all(row["n_active"] == 29 for row in sel["per_step"]) and sel["n_units"] == 144
    assert sel["algorithmic_bytes"] == 250085376
    assert 0 < pc["launch_floor"]["us"] < pc["tiny"]["lump"]["us_cold_l2"] + 4.0
    assert pc["sd3"]["lump"]["back_to_back_rotating_buffers"]["exceeds_4x_l2"] is True
    assert sel["back_to_back_rotating_buffers"]["us_per_step"] > 20.0
    assert set(c["other_workloads_ms_per_layer"]) == {"tiny", "sd3", "qwen768", "temporal"}
