"""Host-side behaviour of bench.py that needs no GPU: the multi-GPU launcher never reports more GPUs
than it has, and the rank count in the environment must agree with --gpus."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env_extra):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env.update(env_extra)
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, env=env, capture_output=True, text=True, timeout=600)


def test_launcher_refuses_more_gpus_than_are_visible():
    res = _run(["--gpus", "2", "--steps", "1"], {"CUDA_VISIBLE_DEVICES": ""})
    assert res.returncode == 2 and "0 CUDA device(s) visible" in res.stderr
    assert res.stdout.strip() == ""                      # no bench line that claims two GPUs


def test_rank_count_from_the_environment_must_match_gpus():
    res = _run(["--gpus", "4", "--steps", "1"], {"CUDA_VISIBLE_DEVICES": "", "WORLD_SIZE": "2", "RANK": "0", "LOCAL_RANK": "0"})
    assert res.returncode != 0 and "must agree" in res.stderr and res.stdout.strip() == ""


def test_one_gpu_without_a_device_fails_loudly():
    res = _run(["--gpus", "1", "--steps", "1"], {"CUDA_VISIBLE_DEVICES": ""})
    assert res.returncode != 0 and "no CPU path" in res.stderr and res.stdout.strip() == ""


def test_reference_arm_other_ranks_do_no_work():
    res = _run(["--impl", "reference", "--gpus", "2", "--steps", "1"], {"WORLD_SIZE": "2", "RANK": "1", "LOCAL_RANK": "1"})
    assert res.returncode == 0 and res.stdout.strip() == ""
