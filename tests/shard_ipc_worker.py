"""Child of tests/test_sharded_gpu.py: one of two ranks that share GPU 0.  Each owns a block of the workers;
peers' message rows are mapped through CUDA IPC; gloo provides the rendezvous and the barriers (host side:
no kernel of one rank ever waits for a kernel of the other).  Each rank checks itself against the oracle."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from oracle import sae_oracle as so                      # noqa: E402
from paper_2008_05823_b200 import binding as sb          # noqa: E402
from paper_2008_05823_b200 import synth                  # noqa: E402
from paper_2008_05823_b200.sharded import sharded_sae    # noqa: E402
from parity_util import assert_same                      # noqa: E402

SIZES = [1, 33, 4096, 5000, 3 * 4096 + 7, 64, 20000]


def run_one(comp, rank):
    K, p, seed = 5, 2, 3
    d = int(np.sum(SIZES))
    scales = synth.tensor_scales(seed, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(seed, d)
    kw = dict(compressor=comp, server_compress=1, mode=so.SAEF, avg_period=p, momentum=0.9, weight_decay=1e-4,
              topk_num=1, topk_den=20)
    orc = so.Oracle(K, SIZES, x0, threads=2, **kw)
    run = sharded_sae(K, SIZES, torch.from_numpy(x0).cuda(), **kw)
    b, c = run.begin, run.count
    cpu = lambda t: t.cpu().numpy()
    for t in range(6):
        g = synth.grads_numpy(seed, t, K, SIZES, scales)
        orc.step(g, 0.1)
        gl = torch.from_numpy(np.ascontiguousarray(g.reshape(K, d)[b:b + c])).cuda()
        run.step(gl, 0.1)
        run.finish()
        e = run.engine
        e.sync()
        tag = f"comp {comp} rank {rank} t={t + 1}"
        assert_same(f"{tag} x", cpu(e.get_params()), orc.get(orc.X))
        assert_same(f"{tag} e_srv", cpu(e.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
        for kl in range(c):
            assert_same(f"{tag} e[{b + kl}]", cpu(e.get_state(sb.STATE_WORKER_ERROR, kl)), orc.get(orc.E, b + kl))
            assert_same(f"{tag} m[{b + kl}]", cpu(e.get_state(sb.STATE_MOMENTUM, kl)), orc.get(orc.M, b + kl))
    run.close()                                           # every reader unmaps before any owner frees


def main():
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    torch.cuda.set_device(0)
    for comp in (so.SIGN, so.TOPK):                       # 1-bit messages, then lists of selected entries
        run_one(comp, rank)
        dist.barrier()
    print("SHARD_OK", rank, flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
