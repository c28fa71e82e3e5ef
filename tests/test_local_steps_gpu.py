"""GPU parity of the local-step extension (Section 2: the model difference communicated every H
iterations) against the CPU oracle: every piece of state after every iteration, the messages after the
communicating ones."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from parity_util import compare_state, compare_server_messages

pytestmark = pytest.mark.gpu

RAGGED = [1, 2, 31, 32, 33, 1000, 4097, 4096, 5000, 8192 + 5, 3 * 4096]


def run_local(K, sizes, comp, steps, H, seed=0, dc=1, mu=0.9, lam=0.0, den=100, lrs=(0.1, 0.05, 0.2), every=1,
              outliers=(0, 1.0)):
    import torch
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(seed, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(seed, d)
    kw = dict(compressor=comp, server_compress=dc, momentum=mu, weight_decay=lam, topk_den=den, local_steps=H)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
    for t in range(steps):
        g = synth.grads_numpy(seed, t, K, sizes, scales, outliers[0], outliers[1])
        lr = lrs[t % len(lrs)]
        orc.step(g, lr)
        gpu.step(torch.from_numpy(g).cuda(), lr)
        if (t + 1) % every == 0 or t == steps - 1:
            tag = f"K={K} comp={comp} H={H} dc={dc} t={t + 1}"
            comm = (t + 1) % H == 0
            compare_state(gpu, orc, comp, check_messages=comm, tag=tag)
            if comm:
                compare_server_messages(gpu, orc, comp, dc, tag=tag)
    assert not orc.range_flag
    gpu.close()


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK, so.IDENTITY])
@pytest.mark.parametrize("H", [1, 2, 3, 4])
@pytest.mark.parametrize("K", [1, 3, 4])
def test_local_steps_ragged(comp, H, K):
    run_local(K, RAGGED, comp, 9, H, den=20, outliers=(66, 100.0), seed=3)


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("mu,lam", [(0.0, 0.0), (0.9, 1e-4), (0.5, 1e-2)])
def test_local_steps_variants(comp, dc, mu, lam):
    """single-way / double-way, no momentum rows (mu = 0), weight decay (the local pass reads x)."""
    run_local(3, RAGGED, comp, 8, 3, dc=dc, mu=mu, lam=lam, den=20, seed=5)


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
def test_local_steps_large_problem(comp):
    """Above the small-problem limit (K * d > 2^24): separate finalize launch, multi-tile server blocks."""
    run_local(2, [5_000_000, 4_500_000, 33, 70_000], comp, 6, 3, every=3, seed=6)


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
@pytest.mark.parametrize("H", [2, 5])
def test_local_steps_graph_replay_without_getters(comp, H):
    """On a side stream the steps replay CUDA graphs (communicating or not is part of the graph key) and the
    server lines of a communicating step stay pending across the local iterations that follow."""
    import torch
    K, sizes, steps = 4, RAGGED, 4 * H + 1
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(7, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(7, d)
    kw = dict(compressor=comp, momentum=0.9, topk_den=20, local_steps=H)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    with torch.cuda.stream(torch.cuda.Stream()):
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
        gs = [torch.from_numpy(synth.grads_numpy(7, t % 3, K, sizes, scales)).cuda() for t in range(3)]
        for t in range(steps):
            orc.step(gs[t % 3].cpu().numpy(), 0.1)
            gpu.step(gs[t % 3], 0.1)
        compare_state(gpu, orc, comp, check_messages=False, tag=f"H={H} after {steps}")
        gpu.close()


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
def test_local_steps_checkpoint_inside_a_round(comp):
    import torch
    K, sizes, H = 3, RAGGED, 4
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(8, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(8, d)
    kw = dict(compressor=comp, momentum=0.9, weight_decay=1e-4, topk_den=20, local_steps=H)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    a = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
    gs = [torch.from_numpy(synth.grads_numpy(8, t, K, sizes, scales)).cuda() for t in range(11)]
    for t in range(6):                                    # 4 communicates; 5 and 6 are local
        orc.step(gs[t].cpu().numpy(), 0.1)
        a.step(gs[t], 0.1)
    blob = a.save_state()
    b = sb.Sae(K, sizes, torch.zeros(d, device="cuda"), **kw)
    b.load_state(blob)
    other = sb.Sae(K, sizes, torch.zeros(d, device="cuda"), **dict(kw, local_steps=2))
    with pytest.raises(sb.SaeError):
        other.load_state(blob)                            # a checkpoint of another period
    other.close()
    for t in range(6, 11):
        orc.step(gs[t].cpu().numpy(), 0.1)
        a.step(gs[t], 0.1)
        b.step(gs[t], 0.1)
    compare_state(a, orc, comp, check_messages=False, tag="continued")
    compare_state(b, orc, comp, check_messages=False, tag="restored")
    a.close(); b.close()


def test_local_steps_argument_checks():
    import torch
    x0 = torch.zeros(100, device="cuda")
    g = torch.zeros(2, 100, device="cuda")
    for kw in (dict(mode=sb.EF), dict(avg_period=3), dict(shard=(0, 1))):
        s = sb.Sae(2, [100], x0, **kw)
        with pytest.raises(sb.SaeError):
            s.set_local_steps(2)
        s.set_local_steps(1) if "shard" not in kw else None
        s.close()
    s = sb.Sae(2, [100], x0)
    with pytest.raises(sb.SaeError):
        s.set_local_steps(0)
    s.step(g, 0.1)
    with pytest.raises(sb.SaeError):
        s.set_local_steps(2)                              # only before the first step
    s.close()
