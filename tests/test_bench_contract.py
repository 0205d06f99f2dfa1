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
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1 and lines[0].startswith("{"), out.stdout[-2000:]     # the JSON line and nothing else
    return json.loads(lines[0])


def test_reference_arm_runs_the_oracle_on_the_host():
    d = run_bench("--impl", "reference", "--workload", "small_f32", "--steps", "2", "--warmup", "3")
    assert BASE <= set(d)
    assert d["impl"] == "reference" and d["unit"] == "params/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"]
    assert d["cpu_baseline"]["single_thread"]["cores"] == 1 and d["cpu_baseline"]["single_thread"]["value"] > 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in d["config"] and "model" not in d["config"]
    assert "wall clock" in d["config"]["timing"] and "CUDA events" not in d["config"]["timing"]


def test_both_arms_time_the_oracle_on_the_same_sample():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.sample_sizes("cfg3_7b_bf16") == (bench.ALL_CORE_SAMPLE, bench.ONE_THREAD_SAMPLE)
    n_all, n_one = bench.sample_sizes("small_f32")
    gs, ds, total, used = bench.oracle_sample("small_f32", n_all)
    assert total == n_all == sum(t.numel() for t in gs) and used == len(gs) == len(ds)
    gs1, _, total1, _ = bench.oracle_sample("small_f32", n_one)
    assert total1 == n_one and all(bool((a[: b.numel()] == b).all()) for a, b in zip(gs, gs1))


def test_gpus_flag_starts_one_rank_per_gpu(tmp_path):
    """--gpus N without a launcher's environment: N workers, each with its own RANK / LOCAL_RANK, the same
    WORLD_SIZE and one free port on 127.0.0.1; the arguments are passed through; a failing rank's
    exit code comes back.  A stub stands in for the worker (no GPU here)."""
    sys.path.insert(0, ROOT)
    import bench
    stub = ("import json, os, sys; "
            "keys = ['RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'LOCAL_WORLD_SIZE', 'MASTER_ADDR', 'MASTER_PORT']; "
            "open(os.path.join(sys.argv[1], os.environ['RANK'] + '.json'), 'w').write("
            "json.dumps({'env': {k: os.environ[k] for k in keys}, 'argv': sys.argv[2:]})); "
            "sys.exit(int(os.environ['RANK']) * int(sys.argv[2] == '--fail'))")
    worker = [sys.executable, "-c", stub, str(tmp_path)]
    assert bench.spawn_ranks(3, ["--gpus", "3", "--steps", "7"], worker=worker) == 0
    seen = [json.load(open(tmp_path / f"{r}.json")) for r in range(3)]
    assert [s["env"]["RANK"] for s in seen] == ["0", "1", "2"]
    assert [s["env"]["LOCAL_RANK"] for s in seen] == ["0", "1", "2"]
    assert {s["env"]["WORLD_SIZE"] for s in seen} == {"3"} and {s["env"]["MASTER_ADDR"] for s in seen} == {"127.0.0.1"}
    ports = {s["env"]["MASTER_PORT"] for s in seen}
    assert len(ports) == 1 and 1024 < int(ports.pop()) < 65536
    assert all(s["argv"] == ["--gpus", "3", "--steps", "7"] for s in seen)
    assert bench.spawn_ranks(2, ["--fail"], worker=worker) == 1
    env = bench.rank_environment(4, 2, 12345, base={"NCCL_DEBUG": "INFO", "RANK": "9"})
    assert env["RANK"] == "2" and env["WORLD_SIZE"] == "4" and env["NCCL_DEBUG"] == "INFO"


def test_gpus_beyond_the_visible_devices_fails_loudly():
    import torch
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "64"], capture_output=True,
                         text=True, timeout=300, cwd=ROOT, env={k: v for k, v in os.environ.items()
                                                                if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")})
    assert out.returncode != 0
    msg = out.stderr
    assert ("CUDA device" in msg) if not torch.cuda.is_available() else ("--gpus 64" in msg)


@pytest.mark.gpu
def test_library_arm_line_on_a_small_list():
    d = run_bench("--workload", "small_bf16", "--also", "small_f32", "--others", "cfg1_flat_f32",
                  "--steps", "3", "--warmup", "3")
    assert BASE <= set(d)
    assert d["n_gpus"] == 1 and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["dtype"] == "bf16 g / f32 d, f64 sums, f32 fma"
    one = d["others"]["cfg1_flat_f32"]
    assert one["params"] == 1 << 20 and one["regime_check"]["regime"] == "project"
    assert abs(one["regime_check"]["cos"] - 0.9) < 0.01 and "launch-bound" in one["note"]
    assert 0 < one["graph_replay_us_per_step"] < 1e3 * one["ms_per_step"] * 1.5
    fa = d["fused_adamw"]
    assert fa["regime"] == "project" and fa["fused_bytes_per_param"] == 34 and fa["roofline"]["bound"] == "hbm"
    assert "fused_adamw_exchange" not in d                 # bf16 g with an f32 snapshot: no exchange mode
    assert d["cpu_baseline"]["single_thread"]["cores"] == 1
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
    d = run_bench("--workload", "small_f32", "--also", "none", "--others", "none", "--steps", "3", "--warmup", "3",
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
    d = run_bench("--workload", "small_f32", "--also", "none", "--others", "none", "--steps", "3", "--warmup", "3",
                  "--sharded", "--no-adamw", "--no-e2e", "--no-cpu-baseline")
    assert d["gpu_launches"] == 3 * d["steps"] and "dp1" in d["config"]["parallelism"]
    assert d["regime_check"]["regime"] == "project" and abs(d["regime_check"]["cos"] - 0.9) < 0.01


@pytest.mark.gpu
def test_sharded_call_sequence_with_the_librarys_own_exchange():
    """Same sequence with --exchange peer: the slot array comes from symmetric memory (a one-rank
    group here), the reduction kernel posts the three sums and a small kernel adds them up."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "small_f32", "--also", "none",
                          "--others", "none", "--steps", "3", "--warmup", "3", "--sharded", "--exchange", "peer",
                          "--no-adamw", "--no-e2e", "--no-cpu-baseline"], capture_output=True, text=True,
                         timeout=900, cwd=ROOT)
    if out.returncode != 0 and "symmetric" in out.stderr.lower():
        pytest.skip("symmetric memory is not available here: " + out.stderr.strip().splitlines()[-1][:200])
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][0])
    assert d["gpu_launches"] == 3 * d["steps"] and "peer stores" in d["config"]["parallelism"]
    assert d["regime_check"]["regime"] == "project" and abs(d["regime_check"]["cos"] - 0.9) < 0.01
