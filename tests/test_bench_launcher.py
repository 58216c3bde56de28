"""`python bench.py --gpus N` must start N ranks by itself (the launcher a torchrun command line would
use), fail when the world that came up is not the one asked for, and print exactly one line from rank
0.  Run here with two gloo ranks and the benchmark's stub step, which needs no GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BENCH = os.path.join(ROOT, "bench.py")


def _env():
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    return env


@pytest.mark.timeout(300)
def test_gpus_flag_starts_that_many_ranks():
    out = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--workload", "stub", "--steps", "3",
                          "--warmup", "1"], env=_env(), capture_output=True, text=True, timeout=280)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["steps"] == 3 and lines[0]["config"]["workload"] == "stub"


@pytest.mark.timeout(120)
def test_world_size_mismatch_is_an_error():
    env = _env()
    env.update(WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")       # a launcher that started one rank only
    out = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--workload", "stub"], env=env,
                         capture_output=True, text=True, timeout=100)
    assert out.returncode != 0 and "--gpus 2" in (out.stderr + out.stdout)


@pytest.mark.timeout(300)
def test_reference_arm_runs_on_rank_zero_only():
    """Under a two-rank launch the reference arm times the oracle on rank 0; the other rank exits 0."""
    out = subprocess.run([sys.executable, BENCH, "--gpus", "2", "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--ref-rows", "4"], env=_env(), capture_output=True, text=True,
                         timeout=280)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["e2e"]["h2d_bytes_per_step"] == 0
    assert lines[0]["value"] > 0 and abs(lines[0]["ms_per_step"] * 1e-3 * lines[0]["value"] - 4) < 1e-6
