"""Seeded random configurations (worker count, tensor list, compressor, schedule, branch, momentum, weight
decay, single/double-way, learning rates), unsharded, sharded and with local steps, against the oracle: every combination the
hand-written cases do not name explicitly still has to give the oracle's bits."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from paper_2008_05823_b200.sharded import worker_range
from parity_util import compare_state, compare_server_messages, assert_same

pytestmark = pytest.mark.gpu

SIZE_POOL = [1, 2, 5, 31, 32, 33, 64, 127, 128, 129, 700, 1000, 4095, 4096, 4097, 5000, 8192, 8192 + 5, 3 * 4096,
             20000, 5 * 4096 + 1]


def draw(case):
    rng = np.random.default_rng(1000 + case)
    cfg = dict(
        K=int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 12, 16, 17, 32, 33])),
        sizes=[int(s) for s in rng.choice(SIZE_POOL, size=int(rng.integers(1, 7)))],
        comp=int(rng.choice([so.SIGN, so.SIGN, so.TOPK, so.IDENTITY])),
        p=int(rng.choice([0, 1, 1, 2, 3, 5])),
        dc=int(rng.integers(0, 2)),
        mode=int(rng.choice([so.EF, so.SAEF])),
        mu=float(rng.choice([0.0, 0.5, 0.9])),
        lam=float(rng.choice([0.0, 1e-4, 1e-2])),
        den=int(rng.choice([2, 10, 100])),
        lrs=[float(x) for x in rng.choice([0.01, 0.05, 0.1, 0.3], size=3)],
        seed=int(rng.integers(0, 1 << 20)),
    )
    return cfg


@pytest.mark.parametrize("case", range(120))
def test_random_configuration(case):
    import torch
    c = draw(case)
    K, sizes = c["K"], c["sizes"]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(c["seed"], len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(c["seed"], d)
    kw = dict(compressor=c["comp"], server_compress=c["dc"], mode=c["mode"], avg_period=c["p"], momentum=c["mu"],
              weight_decay=c["lam"], topk_num=1, topk_den=c["den"])
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
    for t in range(5):
        g = synth.grads_numpy(c["seed"], t, K, sizes, scales, 66, 100.0)
        lr = c["lrs"][t % 3]
        orc.step(g, lr)
        gpu.step(torch.from_numpy(g).cuda(), lr)
        if case % 2 == 0 or t in (1, 4):      # odd cases: no getter between most steps (pending server lines)
            compare_state(gpu, orc, c["comp"], tag=f"case {case} {c} t={t + 1}")
            compare_server_messages(gpu, orc, c["comp"], c["dc"], tag=f"case {case} t={t + 1}")
    assert not orc.range_flag
    gpu.close()


@pytest.mark.parametrize("case", range(40))
def test_random_sharded_configuration(case):
    import torch
    c = draw(100 + case)
    K, sizes = max(2, c["K"]), c["sizes"]
    world = int(np.random.default_rng(case).integers(1, min(K, 4) + 1))
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(c["seed"], len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(c["seed"], d)
    comp = so.TOPK if case % 3 == 2 else so.SIGN
    kw = dict(compressor=comp, server_compress=c["dc"], mode=c["mode"], avg_period=c["p"], momentum=c["mu"],
              weight_decay=c["lam"], topk_num=1, topk_den=c["den"])
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    ranges = [worker_range(K, world, r) for r in range(world)]
    shards = [sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), shard=rg, **kw) for rg in ranges]
    for s in shards:
        for blob in [q.shard_export() for q in shards]:
            s.shard_attach(blob)
    cpu = lambda t: t.cpu().numpy()
    for t in range(5):
        g = synth.grads_numpy(c["seed"], t, K, sizes, scales, 66, 100.0)
        lr = c["lrs"][t % 3]
        orc.step(g, lr)
        gd = torch.from_numpy(g).cuda().view(K, d)
        for s, (b, n) in zip(shards, ranges):
            s.step_begin(gd[b:b + n].contiguous(), lr)
        for s in shards:
            s.step_end()
        for s, (b, n) in zip(shards, ranges):
            s.sync()
            tag = f"sharded case {case} K={K} world={world} {c} t={t + 1} shard@{b}"
            assert_same(f"{tag} x", cpu(s.get_params()), orc.get(orc.X))
            assert_same(f"{tag} e_srv", cpu(s.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
            for kl in range(n):
                assert_same(f"{tag} e[{b + kl}]", cpu(s.get_state(sb.STATE_WORKER_ERROR, kl)), orc.get(orc.E, b + kl))
    for s in shards:
        s.close()


@pytest.mark.parametrize("case", range(40))
def test_random_local_steps_configuration(case):
    """The same draw with the model differences communicated every H iterations (step-ahead branch, p = inf)."""
    import torch
    c = draw(200 + case)
    H = int(np.random.default_rng(case).integers(2, 6))
    K, sizes = c["K"], c["sizes"]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(c["seed"], len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(c["seed"], d)
    kw = dict(compressor=c["comp"], server_compress=c["dc"], momentum=c["mu"], weight_decay=c["lam"], topk_num=1,
              topk_den=c["den"], local_steps=H)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
    for t in range(2 * H + 1):
        g = synth.grads_numpy(c["seed"], t, K, sizes, scales, 66, 100.0)
        lr = c["lrs"][t % 3]
        orc.step(g, lr)
        gpu.step(torch.from_numpy(g).cuda(), lr)
        comm = (t + 1) % H == 0
        if case % 2 == 0 or comm or t == 2 * H:
            compare_state(gpu, orc, c["comp"], check_messages=comm, tag=f"local case {case} H={H} {c} t={t + 1}")
            if comm:
                compare_server_messages(gpu, orc, c["comp"], c["dc"], tag=f"local case {case} t={t + 1}")
    assert not orc.range_flag
    gpu.close()
