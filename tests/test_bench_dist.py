"""Multi-process plumbing of bench.py, on CPU with the gloo backend (world size 2): the path does not
shard, so N > 1 means N independent replicas whose step times are combined as the max over ranks."""
import json
import os
import subprocess
import sys

import pytest

from conftest import free_port

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
got = bench.max_over_ranks(ms)
assert got == 15.0, got
val = bench.whole_job_value(20, got, dist.get_world_size())
assert abs(val - 2 * 20 / 0.015) < 1e-6, val
dist.barrier()
if rank == 0:
    print("OK", got, val)
dist.destroy_process_group()
"""


def _torchrun(args, timeout=300):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", free_port()] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    res = _torchrun([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    assert "OK 15.0" in res.stdout


def test_reference_arm_under_torchrun_prints_one_line_from_rank0():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--workload", "0", "--steps", "2", "--warmup", "1"])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def test_single_process_helpers():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(10, 1000.0, 1) == 10.0
    step, worker, variant = bench.algorithmic_bytes(__import__("paper_2008_05823_b200.configs", fromlist=["x"]).workload(2), 1)
    Wd, d = 16 * 25557032, 25557032
    # (16 workers: the worker pass also writes the sum of the previous step's messages)
    assert step == 12 * Wd + 24 * d and worker == 12 * Wd + 12 * d and variant == "sign_p1_folded16"
