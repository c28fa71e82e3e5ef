"""Rank logic of the sharded run on CPU (gloo, world size 2) with a recording stand-in for the engine: who
owns which workers, that every rank attaches every rank's rows, and the order of begin / barrier / end."""
import os
import subprocess
import sys

import pytest

from conftest import free_port

from paper_2008_05823_b200.sharded import worker_range

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, struct
sys.path.insert(0, {root!r})
import torch.distributed as dist
from paper_2008_05823_b200.sharded import ShardedRun

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
log = []

class Fake:
    def __init__(self, begin, count):
        self.begin, self.count, self.attached = begin, count, []
    def shard_export(self):
        return struct.pack("<ii", self.begin, self.count) + bytes(1016)
    def shard_attach(self, blob):
        assert len(blob) == 1024
        self.attached.append(struct.unpack("<ii", blob[:8]))
    def step_begin(self, g, lr): log.append(("begin", lr))
    def step_end(self): log.append(("end",))
    def shard_detach(self): log.append(("detach",))
    def close(self): log.append(("close",))

def barrier():
    log.append(("barrier",))
    dist.barrier()

K = 5
run = ShardedRun(K, Fake, barrier=barrier)
assert (run.begin, run.count) == ((0, 3) if rank == 0 else (3, 2)), (run.begin, run.count)
assert run.engine.attached == [(0, 3), (3, 2)], run.engine.attached          # every rank's rows, in rank order
assert log == [("barrier",)]
run.step(None, 0.1)
run.step(None, 0.2)
run.close()
assert log == [("barrier",), ("begin", 0.1), ("barrier",), ("end",),          # messages complete before the server pass
               ("barrier",), ("begin", 0.2), ("barrier",), ("end",),          # readers done before rows are rewritten
               ("barrier",), ("detach",), ("barrier",), ("close",)], log      # unmap everywhere before anyone frees
print("OK", rank, flush=True)
dist.destroy_process_group()
"""


def test_worker_range_partitions_the_workers():
    for K in (1, 2, 5, 8, 32, 33):
        for world in range(1, min(K, 8) + 1):
            got = [worker_range(K, world, r) for r in range(world)]
            assert got[0][0] == 0 and sum(c for _, c in got) == K
            for (b0, c0), (b1, _) in zip(got, got[1:]):
                assert b1 == b0 + c0
            assert max(c for _, c in got) - min(c for _, c in got) <= 1
    with pytest.raises(ValueError):
        worker_range(2, 3, 0)
    with pytest.raises(ValueError):
        worker_range(4, 2, 2)


def test_rank_logic_world_size_2(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", free_port(), str(script)]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-3000:]
    assert res.stdout.count("OK") == 2
