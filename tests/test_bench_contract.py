"""The output contract of bench.py: one JSON line with the agreed keys.  The reference arm (the CPU
oracle on a bounded sample) runs anywhere; the GPU arm is checked on a short run."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
             "scaling", "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "cpu_baseline"}


def _run(args, timeout):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True,
                         text=True, timeout=timeout, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_reference_arm_line():
    d = _run(["--impl", "reference", "--steps", "3", "--warmup", "1"], 600)
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["steps"] == 3 and d["warmup"] == 1 and d["n_gpus"] == 1
    assert d["value"] > 0 and d["unit"] == "GB/s" and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("llama2-7b")


@pytest.mark.gpu
def test_gpu_arm_line():
    d = _run(["--steps", "40", "--warmup", "5", "--layers", "2"], 900)
    assert BASE_KEYS | {"roofline", "clocks"} <= set(d)
    assert d["steps"] == 40 and d["warmup"] == 5 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    assert d["gpu_launches"] == 4 * 40 * d["replay_seconds"]["replays"] and d["replay_seconds"]["replays"] >= 50
    assert abs(d["ms_per_step"] - d["replay_seconds"]["median"] * 1e3 / 40) < 1e-9
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.9 < r["traffic"] / r["algorithmic_bytes_per_launch"] < 1.1
    assert abs(r["achieved"] - r["algorithmic_bytes_per_launch"] / r["avg_launch_us"] / 1e3) < 1e-6 * r["achieved"]
    assert len(r["per_position"]) == 4
    assert "NOT more" in d["config"]["l2_policy"]           # two layers (210 MB) do not exceed 2 x L2
    for key in ("config1_single_linear", "config4_70b_mlp", "config5_sweep", "gemm_m2048", "quantize_pack"):
        assert key in d, key
    assert len(d["config4_70b_mlp"]) == 8 and len(d["config5_sweep"]["rows"]) == 66
    assert all("sustained" in g and g["sustained"]["seconds"] >= 2.0 for g in d["gemm_m2048"])
    assert set(d["cpu_baseline"]["phases"]) >= {"quantize_pack_s", "unpack_dequantize_s", "multiply_fp64_s"}
    assert d["e2e"]["h2d_bytes_per_step"] == 46592 and d["e2e"]["d2h_bytes_per_step"] == 84992
    assert 0 < d["e2e"]["value"] < d["value"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["config"]["workload"].startswith("llama2-7b") and "model" not in d["config"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
