"""Multi-GPU runs are independent replicas: what the ranks share is a barrier, the maximum of their times and the
whole-job rate.  These tests run that plumbing as two gloo processes on CPU, and the reference arm of bench.py
under torch.distributed.run with two ranks (rank 0 alone works and prints; the other exits 0 without work)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
from paper_2602_22592_b200 import replicas
reps = replicas.from_env("gloo")
assert reps.world == 2 and reps.backend == "gloo"
reps.barrier()
ms = 10.0 + 5.0 * reps.rank                      # rank 1 is the slow replica
worst = reps.max_over_ranks(ms)
rate = reps.whole_job_rate(8192, worst)
reps.barrier()
if reps.is_root:
    print(json.dumps({{"worst": worst, "rate": rate, "world": reps.world}}))
reps.close()
"""


def _torchrun(args, timeout=600):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(29500 + os.getpid() % 2000)] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    p = _torchrun([str(script)])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["world"] == 2
    assert out["worst"] == 15.0                     # the maximum over ranks, not the mean or rank 0's own
    assert out["rate"] == pytest.approx(2 * 8192 / 15.0e-3)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_2602_22592_b200 import replicas
    env = {k: os.environ.pop(k) for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE") if k in os.environ}
    try:
        reps = replicas.from_env("gloo")
        assert (reps.rank, reps.world, reps.backend) == (0, 1, None)
        reps.barrier()
        assert reps.max_over_ranks(3.5) == 3.5
        assert reps.whole_job_rate(100, 2.0) == pytest.approx(100 / 2.0e-3)
        reps.close()
    finally:
        os.environ.update(env)


def test_reference_arm_under_two_ranks_prints_once():
    p = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--cpu-tokens", "32"])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0


def test_gpus_flag_without_torchrun_launches_the_ranks_itself():
    # `python bench.py --gpus 2 ...` from a plain shell: the script starts two ranks of its own command line under
    # torch.distributed.run (rendezvous on 127.0.0.1) instead of silently running one
    env = dict(os.environ, OMP_NUM_THREADS="2")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    p = subprocess.run([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "0", "--cpu-tokens", "32"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["steps"] == 2
