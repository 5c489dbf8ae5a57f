"""`python bench.py --gpus N` outside torchrun must start N ranks itself (and refuse when the box
has fewer GPUs) instead of timing one GPU and labelling it N."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*argv, env_drop=("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")):
    env = {k: v for k, v in os.environ.items() if k not in env_drop}
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], env=env, capture_output=True,
                          text=True, timeout=300)


def test_gpus_2_spawns_two_ranks_that_both_report():
    p = _run("--gpus", "2", "--impl", "stub", "--steps", "5", "--warmup", "1")
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, "exactly one JSON line (rank 0's): %r" % p.stdout
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["ranks_reported"] == [0, 1] and rec["steps"] == 5


def test_gpus_2_on_a_box_without_two_gpus_fails_with_a_message():
    import torch

    if torch.cuda.is_available() and torch.cuda.device_count() >= 2:
        import pytest

        pytest.skip("this box has two GPUs")
    p = _run("--gpus", "2", "--steps", "5", "--warmup", "1")
    assert p.returncode != 0
    assert "CUDA device" in p.stderr and "--gpus 2" in p.stderr
    assert not [l for l in p.stdout.splitlines() if l.startswith("{")], "no result line may be printed"


def test_reference_arm_runs_on_rank_0_only_and_prints_the_shared_config_keys():
    sys.path.insert(0, ROOT)
    import bench

    keys = bench.config_keys()
    assert keys["workload"] == "decode_b64" and set(keys) == {"workload", "B_per_gpu", "Hqk", "Hv", "d", "state", "l2"}
