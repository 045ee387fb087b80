"""The N>1 path of bench.py on CPU: two gloo ranks run its rank bookkeeping (max over ranks of
the per-rank device time, whole-job aggregate, rank 0 alone reporting) and the reference arm
(rank 0 alone runs and prints; the other rank exits 0 without work)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# rank r "measured" (r + 1) * 10 ms for its own replica of the workload
ms = bench.max_over_ranks(10.0 * (rank + 1), world, torch.device("cpu"))
val = bench.whole_job_value(world, tokens=1000, n_layers=4, ms_step=ms)
if rank == 0:
    print(json.dumps({{"ms": ms, "value": val, "world": world}}))
dist.destroy_process_group()
"""


def _torchrun(args, port):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    return subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    r = _torchrun([str(script)], 29611)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone reports
    out = json.loads(lines[0])
    assert out["world"] == 2 and out["ms"] == pytest.approx(20.0)          # the slower rank's time
    # weak scaling: both ranks processed tokens * layers in that time
    assert out["value"] == pytest.approx(2 * 1000 * 4 / 20.0e-3)


def test_reference_arm_under_torchrun_prints_once():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                   "--config", "tiny"], 29612)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["cpu_baseline"]["kind"] == "oracle"
    assert out["e2e"]["h2d_bytes_per_step"] == 0 and out["value"] > 0
