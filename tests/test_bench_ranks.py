"""The multi-rank logic of bench.py on CPU: two gloo ranks agree on the slowest rank's time, the
whole-job rate counts every replica, and the reference arm prints one line from rank 0 only."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["EF21_ROOT"])
import torch, torch.distributed as dist
import bench
rank, _, world = bench.dist_env()
dist.init_process_group("gloo")
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
rate = bench.whole_job_rate(2000, world, ms)
# one os.write per rank: two ranks' lines never share a line of the merged output
os.write(1, (json.dumps({"rank": rank, "world": world, "ms": ms, "rate": rate}) + "\n").encode())
dist.destroy_process_group()
"""


def _launch(world, argv, env_extra=None, timeout=300):
    env = dict(os.environ, EF21_ROOT=ROOT, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
           "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000)] + argv
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def _json_lines(text):
    out = []
    for ln in text.splitlines():
        ln = ln.strip()
        if ln.startswith("{") and ln.endswith("}"):
            out.append(json.loads(ln))
    return out


def test_two_ranks_take_the_slowest_time(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    p = _launch(2, [str(script)])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = sorted(_json_lines(p.stdout), key=lambda r: r["rank"])
    assert [r["rank"] for r in lines] == [0, 1]
    for r in lines:
        assert r["world"] == 2
        assert r["ms"] == 15.0                                  # max over ranks, on every rank
        assert r["rate"] == pytest.approx(2 * 2000 / 15e-3)      # both replicas' iterations over the slowest time


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_rate(100, 1, 50.0) == pytest.approx(2000.0)


def test_reference_arm_prints_once_under_two_ranks():
    p = _launch(2, [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "20", "--warmup", "3"])
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [r for r in _json_lines(p.stdout) if r.get("impl") == "reference"]
    assert len(lines) == 1
    r = lines[0]
    assert r["n_gpus"] == 2 and r["steps"] == 20 and r["cpu_baseline"]["kind"] == "oracle"
    assert r["e2e"]["h2d_bytes_per_step"] == 0 and r["value"] > 0
