"""Sharded operation (the workers of Algorithm 1 spread over several handles) against the CPU oracle.

* Shards of one process on one stream: every shard must hold the oracle's x and server error bit for bit,
  and its own workers' momentum, error, scales and sign words -- the server pass reads all K messages in
  place through the row tables, in k order.
* Two processes on ONE GPU (gloo for the rendezvous and the barriers): the same through CUDA IPC mappings.
  No kernel waits on another: the order between the ranks is enforced on the host.
"""
import os
import subprocess
import sys

import numpy as np
import pytest

from conftest import free_port

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from paper_2008_05823_b200.sharded import worker_range
from parity_util import assert_same

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SIZES = [1, 33, 4096, 5000, 3 * 4096 + 7, 64, 20000]


def compare_shard(shard, begin, orc, dc, tag):
    cpu = lambda t: t.cpu().numpy()
    shard.sync()
    assert shard.iteration == orc.iteration
    assert_same(f"{tag} x", cpu(shard.get_params()), orc.get(orc.X))
    assert_same(f"{tag} e_srv", cpu(shard.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
    for kl in range(shard.K):
        k = begin + kl
        assert_same(f"{tag} m[{k}]", cpu(shard.get_state(sb.STATE_MOMENTUM, kl)), orc.get(orc.M, k))
        assert_same(f"{tag} e[{k}]", cpu(shard.get_state(sb.STATE_WORKER_ERROR, kl)), orc.get(orc.E, k))
        assert_same(f"{tag} step_ahead[{k}]", cpu(shard.get_step_ahead(kl)), orc.step_ahead(k))
        if orc.iteration:
            assert_same(f"{tag} scales[{k}]", cpu(shard.get_state(sb.STATE_WORKER_SCALES, kl)), orc.get(orc.SCALES, k))
            assert_same(f"{tag} words[{k}]", cpu(shard.get_state(sb.STATE_WORKER_WORDS, kl)).view(np.uint32),
                        so.pack_signs(orc.get(orc.DELTA, k), orc.sizes))
    if dc and orc.iteration:
        assert_same(f"{tag} scales_srv", cpu(shard.get_state(sb.STATE_SERVER_SCALES)), orc.get(orc.SCALES_SRV))
        assert_same(f"{tag} words_srv", cpu(shard.get_state(sb.STATE_SERVER_WORDS)).view(np.uint32),
                    so.pack_signs(orc.get(orc.DELTA_SRV), orc.sizes))


@pytest.mark.parametrize("K,world", [(4, 2), (3, 2), (5, 3), (4, 4), (2, 1)])
@pytest.mark.parametrize("p", [0, 1, 3])
@pytest.mark.parametrize("dc,mode,lam", [(1, so.SAEF, 0.0), (0, so.EF, 1e-4)])
def test_shards_in_one_process_match_the_oracle(K, world, p, dc, mode, lam):
    import torch
    d = int(np.sum(SIZES))
    seed = 11
    scales = synth.tensor_scales(seed, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(seed, d)
    kw = dict(compressor=so.SIGN, server_compress=dc, mode=mode, avg_period=p, momentum=0.9, weight_decay=lam)
    orc = so.Oracle(K, SIZES, x0, threads=4, **kw)
    x0d = torch.from_numpy(x0).cuda()
    ranges = [worker_range(K, world, r) for r in range(world)]
    shards = [sb.Sae(K, SIZES, x0d, shard=rg, **kw) for rg in ranges]
    blobs = [s.shard_export() for s in shards]
    for s in shards:
        for b in blobs:
            s.shard_attach(b)
    lrs = [0.1, 0.05, 0.2]
    for t in range(7):
        g = synth.grads_numpy(seed, t, K, SIZES, scales)
        orc.step(g, lrs[t % 3])
        gd = torch.from_numpy(g).cuda().view(K, d)
        for s, (b, c) in zip(shards, ranges):
            s.step_begin(gd[b:b + c].contiguous(), lrs[t % 3])
        for s in shards:                     # same stream: every begin is ordered before every end
            s.step_end()
        for s, (b, c) in zip(shards, ranges):
            compare_shard(s, b, orc, dc, tag=f"K={K} world={world} p={p} shard@{b} t={t + 1}")
    for s in shards:
        s.close()


def test_sharded_handle_checks_its_arguments():
    import torch
    d = int(np.sum(SIZES))
    x0 = torch.zeros(d, device="cuda")
    with pytest.raises(sb.SaeError):
        sb.Sae(4, SIZES, x0, compressor=so.IDENTITY, shard=(0, 2))      # the identity compressor is not sharded
    with pytest.raises(sb.SaeError):
        sb.Sae(4, SIZES, x0, shard=(3, 2))                               # rows beyond K
    a = sb.Sae(4, SIZES, x0, shard=(0, 2))
    g = torch.zeros(2 * d, device="cuda")
    with pytest.raises(sb.SaeError):
        a.step_begin(g, 0.1)                                             # peers not attached yet
    with pytest.raises(sb.SaeError):
        a.step(g, 0.1)                                                   # the unsharded step is refused
    blob = a.shard_export()
    a.shard_attach(blob)
    with pytest.raises(sb.SaeError):
        a.shard_attach(blob)                                             # rows attached twice
    with pytest.raises(sb.SaeError):
        a.step_end()                                                     # no step in flight
    other = sb.Sae(4, SIZES + [5], torch.zeros(d + 5, device="cuda"), shard=(2, 2))
    with pytest.raises(sb.SaeError):
        a.shard_attach(other.shard_export())                             # a different parameter list
    # rows of the same process on a device this handle's device cannot reach (here: one that does not exist):
    # refused on the host, nothing attached, no kernel ever sees the pointers
    peer = sb.Sae(4, SIZES, x0, shard=(2, 2))
    foreign = bytearray(peer.shard_export())
    assert int.from_bytes(foreign[12:16], "little", signed=True) == torch.cuda.current_device()
    foreign[12:16] = int(torch.cuda.device_count()).to_bytes(4, "little", signed=True)
    with pytest.raises(sb.SaeError) as err:
        a.shard_attach(bytes(foreign))
    assert err.value.status == sb.ERR_INVALID_ARG
    with pytest.raises(sb.SaeError):
        a.step_begin(g, 0.1)                                             # still not every worker attached
    a.shard_attach(peer.shard_export())                                  # the untouched blob is accepted
    a.close()
    peer.close()
    other.close()


def test_two_processes_on_one_gpu_through_ipc():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="2")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", free_port(), os.path.join(ROOT, "tests", "shard_ipc_worker.py")]
    res = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, (res.stdout[-2000:], res.stderr[-3000:])
    assert res.stdout.count("SHARD_OK") == 2, res.stdout[-2000:]


def test_unsharded_reference_run_on_the_same_sizes():
    from test_parity_gpu import run_pair
    run_pair(4, SIZES, so.SIGN, 5, p=3, seed=11)


def test_config2_fullsize_shards_equal_the_single_handle():
    """Config 2 at full size (16 workers x 25.6 M parameters): three shards (6 + 5 + 5 workers) against the
    unsharded handle -- itself checked against the oracle at this size elsewhere -- on every piece of state,
    for a schedule with and one without error averaging."""
    import torch
    from paper_2008_05823_b200 import configs
    w = configs.workload(2)
    K, sizes, d = w.num_workers, w.tensor_sizes, w.d
    scales = synth.workload_scales(w, 0)
    gen = synth.DeviceGenerator(sizes, scales)
    x0 = torch.empty(d, device="cuda")
    gen.x0(x0, 0)
    g = torch.empty(K, d, device="cuda")
    for p, steps in ((0, 4), (3, 7)):
        kw = dict(compressor=so.SIGN, avg_period=p, momentum=w.momentum, weight_decay=w.weight_decay)
        one = sb.Sae(K, sizes, x0, **kw)
        ranges = [worker_range(K, 3, r) for r in range(3)]
        shards = [sb.Sae(K, sizes, x0, shard=rg, **kw) for rg in ranges]
        blobs = [s.shard_export() for s in shards]
        for s in shards:
            for b in blobs:
                s.shard_attach(b)
        for t in range(steps):
            gen.grads(g, K, 0, t, w.outlier_per_65536, w.outlier_mult)
            one.step(g, w.lr)
            for s, (b, c) in zip(shards, ranges):
                s.step_begin(g[b:b + c], w.lr)
            for s in shards:
                s.step_end()
        one.sync()
        x_ref, es_ref = one.get_params(), one.get_state(sb.STATE_SERVER_ERROR)
        for s, (b, c) in zip(shards, ranges):
            s.sync()
            assert torch.equal(s.get_params().view(torch.int32), x_ref.view(torch.int32)), f"p={p} x of shard@{b}"
            assert torch.equal(s.get_state(sb.STATE_SERVER_ERROR).view(torch.int32), es_ref.view(torch.int32))
            for kl in (0, c - 1):
                for which in (sb.STATE_MOMENTUM, sb.STATE_WORKER_ERROR, sb.STATE_WORKER_WORDS, sb.STATE_WORKER_SCALES):
                    a, r = s.get_state(which, kl), one.get_state(which, b + kl)
                    assert torch.equal(a.view(torch.int32), r.view(torch.int32)), f"p={p} state {which} worker {b + kl}"
            s.close()
        one.close()


NCCL_WORKER = r"""
import os, sys
import numpy as np, torch, torch.distributed as dist
sys.path.insert(0, {root!r}); sys.path.insert(0, os.path.join({root!r}, "tests"))
from oracle import sae_oracle as so
from paper_2008_05823_b200 import synth
from paper_2008_05823_b200.sharded import sharded_sae
os.environ.setdefault("MASTER_ADDR", "127.0.0.1"); os.environ.setdefault("MASTER_PORT", {port!r})
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
sizes = [33, 4096, 5000]
K, d = 3, sum(sizes)
scales = synth.tensor_scales(1, len(sizes), -4.0, -1.0)
x0 = synth.x0_numpy(1, d)
orc = so.Oracle(K, sizes, x0, compressor=so.SIGN, avg_period=2, momentum=0.9)
run = sharded_sae(K, sizes, torch.from_numpy(x0).cuda(), avg_period=2, momentum=0.9)
assert run._flag is not None                      # the stream-ordered barrier is in use
for t in range(4):
    g = synth.grads_numpy(1, t, K, sizes, scales)
    orc.step(g, 0.1)
    run.step(torch.from_numpy(g).cuda(), 0.1)
run.finish()
torch.cuda.synchronize()
assert np.array_equal(run.engine.get_params().cpu().numpy().view(np.uint32), orc.get(orc.X).view(np.uint32))
run.close()
dist.destroy_process_group()
print("NCCL_OK")
"""


def test_stream_ordered_barrier_with_the_nccl_backend(tmp_path):
    """World size 1 (this box has one GPU): the NCCL code path of the rank logic -- all-gather of the row
    descriptions, the one-element all-reduce as the stream-ordered barrier, orderly shutdown."""
    script = tmp_path / "nccl_worker.py"
    script.write_text(NCCL_WORKER.format(root=ROOT, port=free_port()))
    res = subprocess.run([sys.executable, str(script)], cwd=ROOT, capture_output=True, text=True, timeout=600,
                         env=dict(os.environ, OMP_NUM_THREADS="2"))
    assert res.returncode == 0, (res.stdout[-1000:], res.stderr[-3000:])
    assert "NCCL_OK" in res.stdout


@pytest.mark.parametrize("world", [1, 2, 3])
def test_error_averaging_by_allreduce(world):
    """The all-reduce form of the error averaging (Section 3.2).  One shard: the sum is the shard's own ordered
    sum, so everything stays bit-exact.  Several shards: the partial sums are added in another order than
    k = 0..K-1, so the averaged error matches the oracle to fp32 rounding (and everything that does not yet
    depend on it, bit for bit)."""
    import torch
    K, p = 5, 3
    d = int(np.sum(SIZES))
    scales = synth.tensor_scales(2, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(2, d)
    kw = dict(compressor=so.SIGN, avg_period=p, momentum=0.9, weight_decay=1e-4)
    orc = so.Oracle(K, SIZES, x0, threads=4, **kw)
    ranges = [worker_range(K, world, r) for r in range(world)]
    shards = [sb.Sae(K, SIZES, torch.from_numpy(x0).cuda(), shard=rg, **kw) for rg in ranges]
    for s in shards:
        for blob in [q.shard_export() for q in shards]:
            s.shard_attach(blob)
        s.shard_set_avg_mode(True)
    steps = 6 if world == 1 else 2            # the first averaging is owed after step 2 ((t + 2) mod 3 = 0 at t = 1)
    for t in range(steps):
        g = synth.grads_numpy(2, t, K, SIZES, scales)
        orc.step(g, 0.1)
        gd = torch.from_numpy(g).cuda().view(K, d)
        for s, (b, c) in zip(shards, ranges):
            s.step_begin(gd[b:b + c].contiguous(), 0.1)
        for s in shards:
            s.step_end()
        due = [s.avg_due for s in shards]
        assert all(due) == any(due) and due[0] == ((t + 2) % p == 0)
        if due[0]:
            with pytest.raises(sb.SaeError):
                shards[0].step_begin(gd[:ranges[0][1]].contiguous(), 0.1)      # refused while the sum is owed
            total = None
            for s in shards:                                                    # the "all-reduce", in rank order
                part = s.avg_local_sum()
                total = part if total is None else total + part
            for s in shards:
                s.avg_set(total)
        for s, (b, c) in zip(shards, ranges):
            s.sync()
            got_x = s.get_params().cpu().numpy()
            got_e = s.get_state(sb.STATE_WORKER_ERROR, 0).cpu().numpy()
            if world == 1:
                assert_same(f"t={t + 1} x", got_x, orc.get(orc.X))
                assert_same(f"t={t + 1} e", got_e, orc.get(orc.E, b))
            else:
                assert_same(f"t={t + 1} x", got_x, orc.get(orc.X))             # does not depend on the average yet
                # a mean of K terms of mixed sign: a few roundings of the largest term, absolute
                exp_e = orc.get(orc.E, b)
                np.testing.assert_allclose(got_e, exp_e, rtol=2e-6, atol=2.0 ** -22 * float(np.abs(exp_e).max()))
    for s in shards:
        s.close()



def compare_topk_shard(shard, begin, orc, dc, tag):
    cpu = lambda t: t.cpu().numpy()
    from parity_util import mask_words
    shard.sync()
    assert_same(f"{tag} x", cpu(shard.get_params()), orc.get(orc.X))
    assert_same(f"{tag} e_srv", cpu(shard.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
    for kl in range(shard.K):
        k = begin + kl
        if shard.keeps_momentum:
            assert_same(f"{tag} m[{k}]", cpu(shard.get_state(sb.STATE_MOMENTUM, kl)), orc.get(orc.M, k))
        assert_same(f"{tag} e[{k}]", cpu(shard.get_state(sb.STATE_WORKER_ERROR, kl)), orc.get(orc.E, k))
        assert_same(f"{tag} tau[{k}]", cpu(shard.get_state(sb.STATE_WORKER_TAU, kl)).view(np.uint32).astype(np.uint64),
                    orc.tau(k))
    if dc:
        assert_same(f"{tag} tau_srv", cpu(shard.get_state(sb.STATE_SERVER_TAU)).view(np.uint32).astype(np.uint64),
                    orc.tau(-1))
        assert_same(f"{tag} mask_srv", cpu(shard.get_state(sb.STATE_SERVER_MASK)).view(np.uint32),
                    mask_words(orc.get(orc.C_DELTA_SRV) != 0, orc.sizes))


@pytest.mark.parametrize("K,world", [(4, 2), (3, 2), (5, 3), (2, 1)])
@pytest.mark.parametrize("p", [0, 1, 3])
@pytest.mark.parametrize("dc,mode,lam,den", [(1, so.SAEF, 0.0, 100), (0, so.EF, 1e-4, 10)])
def test_topk_shards_in_one_process_match_the_oracle(K, world, p, dc, mode, lam, den):
    """Top-K messages as lists of selected entries, added in k order by every shard."""
    import torch
    d = int(np.sum(SIZES))
    seed = 13
    scales = synth.tensor_scales(seed, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(seed, d)
    kw = dict(compressor=so.TOPK, server_compress=dc, mode=mode, avg_period=p, momentum=0.9, weight_decay=lam,
              topk_num=1, topk_den=den)
    orc = so.Oracle(K, SIZES, x0, threads=4, **kw)
    ranges = [worker_range(K, world, r) for r in range(world)]
    shards = [sb.Sae(K, SIZES, torch.from_numpy(x0).cuda(), shard=rg, **kw) for rg in ranges]
    blobs = [s.shard_export() for s in shards]
    for s in shards:
        for b in blobs:
            s.shard_attach(b)
    for t in range(7):
        g = synth.grads_numpy(seed, t, K, SIZES, scales, 66, 100.0)
        orc.step(g, 0.1)
        gd = torch.from_numpy(g).cuda().view(K, d)
        for s, (b, c) in zip(shards, ranges):
            s.step_begin(gd[b:b + c].contiguous(), 0.1)
        for s in shards:
            s.step_end()
        for s, (b, c) in zip(shards, ranges):
            compare_topk_shard(s, b, orc, dc, tag=f"topk K={K} world={world} p={p} shard@{b} t={t + 1}")
    for s in shards:
        s.close()


def test_topk_shards_with_overflowing_lists():
    """Gradients of one constant magnitude: every entry ties the k-th magnitude, so all n are selected and the
    lists overflow their regions; the readers then take that worker's stored row with its threshold."""
    import torch
    sizes = [20000, 64, 9000]
    K, d = 3, sum(sizes)
    x0 = np.zeros(d, dtype=np.float32)
    kw = dict(compressor=so.TOPK, avg_period=2, momentum=0.0, topk_num=1, topk_den=100)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    ranges = [(0, 2), (2, 1)]
    shards = [sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), shard=rg, **kw) for rg in ranges]
    for s in shards:
        for blob in [q.shard_export() for q in shards]:
            s.shard_attach(blob)
    rng = np.random.default_rng(3)
    for t in range(4):
        g = (rng.integers(0, 2, size=(K, d)).astype(np.float32) * 2 - 1) * np.float32(0.25)
        orc.step(g.ravel(), 0.5)
        gd = torch.from_numpy(g).cuda()
        for s, (b, c) in zip(shards, ranges):
            s.step_begin(gd[b:b + c].contiguous(), 0.5)
        for s in shards:
            s.step_end()
        for s, (b, c) in zip(shards, ranges):
            compare_topk_shard(s, b, orc, 1, tag=f"overflow t={t + 1} shard@{b}")
    for s in shards:
        s.close()
