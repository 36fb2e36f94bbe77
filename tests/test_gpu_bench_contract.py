"""The benchmark's one-line JSON contract, checked on the tiny workload."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_bench_prints_one_json_line_with_every_key():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny", "--steps", "20",
                          "--warmup", "3"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    r = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
                "roofline", "cpu_baseline", "remap", "timed_repeats", "ms_per_step_min", "ms_per_step_max",
                "kimi_remap_sweep"):
        assert key in r, key
    assert r["value"] > 0 and r["steps"] == 20 and r["n_gpus"] == 1 and r["scaling"] == "weak"
    assert r["vs_baseline"] is None and r["data"] == "synthetic" and "workload" in r["config"]
    assert r["gpu_launches"] >= 3 * 20
    rf = r["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    assert rf["traffic"] is None                       # ncu traffic figures belong to the DSv3 shape only
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["cores"] == 1
    assert r["cpu_baseline"]["host_cores"] >= 1 and "cpu_model" in r["cpu_baseline"]
    assert r["timed_repeats"] >= 3 and r["clocks"]["samples"] >= 5
    assert r["kimi_remap_sweep"] is None               # part of the default (DSv3-shaped) run only
    assert "eager leg" in rf["per_kernel_source"]
    assert r["e2e"]["h2d_bytes_per_step"] > 0 and r["e2e"]["d2h_bytes_per_step"] > 0
    assert r["remap"]["first_step_matches_oracle"] is True and r["remap"]["graph_recaptured"] is False


@pytest.mark.gpu
def test_exchange_path_of_the_benchmark_runs_as_a_group_of_one():
    # the code `bench.py --gpus N` runs on every rank (NCCL, symmetric memory, moe_ep_*), here with N = 1
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--exchange", "--workload", "mixtral",
                          "--tokens", "512", "--steps", "10", "--warmup", "3"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT,
                         env={k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")})
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["n_gpus"] == 1 and r["value"] > 0 and r["e2e"]["value"] > 0
    assert r["config"]["T_per_gpu"] == 512 and r["config"]["slots_per_gpu"] == 8
    assert r["independent_replicas"]["value"] > 0 and r["gpu_launches"] >= 40
