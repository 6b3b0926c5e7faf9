"""The benchmark's reference arm runs on the host cores alone: check the JSON line it prints
against the keys the two arms share (the CUDA arm's line is checked on a GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
COMMON = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
          "scaling", "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline"}


def _env(extra=None):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env.update(extra or {})
    return env


def _run(*args, env=None):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True,
                         text=True, timeout=600, env=_env(env))
    assert out.returncode == 0, out.stderr[-2000:]
    return out.stdout.strip().splitlines()


def test_reference_arm_line():
    lines = _run("--impl", "reference", "--workload", "tiny", "--steps", "2", "--warmup", "1")
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert COMMON <= set(d) and d["impl"] == "reference"
    assert d["unit"] == "tokens/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["config"]["workload"] == "tiny" and d["steps"] == 2 and d["warmup"] == 1
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}


def test_reference_arm_with_gpus_flag_prints_one_line_for_the_whole_job():
    # started plainly (no launcher): --gpus N is honoured, the oracle still runs once, on rank 0
    lines = _run("--impl", "reference", "--gpus", "2", "--workload", "tiny", "--steps", "1", "--warmup", "0")
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["impl"] == "reference"
    host = d["cpu_baseline"]["host"]
    assert host["nproc"] >= 1 and "cpu_model" in host and "ram_gb" in host


def test_cuda_arm_refuses_more_gpus_than_the_machine_shows():
    import torch
    n = torch.cuda.device_count() + 1 if torch.cuda.is_available() else 2
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(n), "--workload",
                          "tiny"], capture_output=True, text=True, timeout=600, env=_env())
    assert out.returncode != 0 and out.stdout.strip() == ""
    assert f"--gpus {n}" in out.stderr and "visible" in out.stderr


def test_reference_arm_is_silent_on_other_ranks():
    lines = _run("--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0",
                 env={"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"})
    assert lines == []


@pytest.mark.gpu
def test_cuda_arm_line():
    lines = _run("--workload", "tiny", "--steps", "4", "--warmup", "3")
    d = json.loads(lines[-1])
    assert COMMON <= set(d) and "impl" not in d
    assert {"clocks", "gpu_launches", "roofline"} <= set(d)
    assert d["gpu_launches"] == 3 * 4 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["e2e"]["value"] < d["value"]
    assert d["cpu_baseline"]["kind"] == "oracle"
