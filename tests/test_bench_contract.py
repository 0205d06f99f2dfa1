"""bench.py prints one JSON line with the agreed keys (reference arm on CPU;
the library's arm on a GPU, on a small list so that it ends in seconds)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
        "scaling", "vs_baseline", "dtype", "data", "config", "e2e"}


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True,
                         text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_runs_the_oracle_on_the_host():
    d = run_bench("--impl", "reference", "--workload", "small_f32", "--steps", "2", "--warmup", "3")
    assert BASE <= set(d)
    assert d["impl"] == "reference" and d["unit"] == "params/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in d["config"] and "model" not in d["config"]


@pytest.mark.gpu
def test_library_arm_line_on_a_small_list():
    d = run_bench("--workload", "small_bf16", "--also", "small_f32", "--steps", "3", "--warmup", "3")
    assert BASE <= set(d)
    assert d["n_gpus"] == 1 and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["gpu_launches"] == 2 * d["steps"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["regime_check"]["regime"] == "project" and abs(d["regime_check"]["cos"] - 0.95) < 0.01
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > d["e2e"]["h2d_bytes_per_step"]
    assert d["cpu_baseline"]["kind"] == "oracle"
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    assert d["also"]["regime_check"]["regime"] == "project"
    assert d["unchanged_regime"]["regime"] == "violation"
    # the float32 list also reports exchange mode: fewer bytes per parameter, same regimes
    x = d["also"]["exchange_mode"]
    assert x["project"]["regime"] == "project" and x["project"]["bytes_per_param"] == 20
    assert x["unchanged"]["regime"] == "violation" and x["unchanged"]["bytes_per_param"] == 8
    assert x["project"]["roofline"]["bound"] == "hbm"


@pytest.mark.gpu
def test_fused_adamw_legs_on_a_small_list():
    d = run_bench("--workload", "small_f32", "--also", "none", "--steps", "3", "--warmup", "3", "--adamw",
                  "--no-e2e", "--no-cpu-baseline")
    assert d["fused_adamw"]["regime"] == "project" and d["fused_adamw"]["fused_bytes_per_param"] == 36
    assert d["fused_adamw_exchange"]["regime"] == "project"
    assert d["fused_adamw_exchange"]["fused_bytes_per_param"] == 32
    assert d["fused_adamw"]["applied_steps"] == d["fused_adamw_exchange"]["applied_steps"] > 0
    assert d["exchange_mode"]["project"]["regime"] == "project"


@pytest.mark.gpu
def test_sharded_call_sequence_with_a_one_rank_nccl_group():
    """The multi-GPU call sequence (local sums, NCCL all-reduce of three doubles, decision,
    projection) on one GPU: same numbers as the unsharded line, three launches per step."""
    d = run_bench("--workload", "small_f32", "--also", "none", "--steps", "3", "--warmup", "3", "--sharded",
                  "--no-e2e", "--no-cpu-baseline")
    assert d["gpu_launches"] == 3 * d["steps"]
    assert d["regime_check"]["regime"] == "project" and abs(d["regime_check"]["cos"] - 0.9) < 0.01
