"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job throughput,
and the reference arm that only rank 0 runs."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
# rank r pretends its step took 1 + r ms and its kernels (2 + r, 3 - r) ms
got = bench.max_over_ranks([1.0 + rank, 2.0 + rank, 3.0 - rank], dist, "cpu")
dist.barrier()
if rank == 0:
    print(json.dumps({"max": got, "value": bench.job_throughput(1000000, world, got[0]), "world": world}))
dist.destroy_process_group()
"""


def test_two_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, REPO_ROOT=ROOT)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["world"] == 2 and res["max"] == [2.0, 3.0, 3.0]
    # two replicas of 4 MB in 2 ms
    assert res["value"] == pytest.approx(2 * 4e6 / 2e-3 / 1e9)


def test_reference_arm_prints_one_line_on_rank_0_only():
    base = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0",
            "--workload", "cfg1_act", "--reference-sample", str(1 << 16), "--gpus", "2"]
    out0 = subprocess.run(base, env=dict(os.environ, RANK="0", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    out1 = subprocess.run(base, env=dict(os.environ, RANK="1", WORLD_SIZE="2"), capture_output=True, text=True, timeout=300)
    assert out0.returncode == 0 and out1.returncode == 0
    assert out1.stdout.strip() == ""
    line = json.loads(out0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "cfg1_act"


def test_algorithmic_bytes_per_element():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.algorithmic_bytes(4096, 4096, 8) == 4096 * (4 + 1 + 8 / 4096)
    assert bench.algorithmic_bytes(1 << 20, 1024, 2) == (1 << 20) * (4 + 0.25 + 8 / 1024)
