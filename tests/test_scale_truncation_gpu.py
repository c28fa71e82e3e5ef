"""Eq. 2's scale ||v||_1 / n on the GPU where the reading of "exact sum -> double" matters: tensors whose exact
fixed-point L1 sum gives one float when its bits below the top 53 are dropped (the reading taken, on both
sides) and another when they are rounded in.  The kernels must follow the oracle -- and the exact rational
arithmetic of tests/scale_cases.py -- bit for bit."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
import scale_cases

pytestmark = pytest.mark.gpu

CASES = [(8, 60), (8, 90), (4096, 62), (5000, 70), (3 * 4096 + 7, 93), (1 << 20, 66)]


def _tensors(seed):
    return [scale_cases.discriminating_tensor(n, top, seed=seed + n) for n, top in CASES]


@pytest.mark.parametrize("filler", [0, (1 << 24) + 4096 + 5])
def test_worker_and_server_scales_follow_the_truncating_reading(filler):
    """One worker, mu = 0, lr = 1, zero state: the first step compresses exactly the gradient, so the worker
    scales are C(v) of each tensor.  Without the filler tensor the problem is small (the server pass forms
    the scales from the records itself), with it the finalize kernel does."""
    import torch
    vs = _tensors(3)
    sizes = [v.size for v in vs] + ([filler] if filler else [])
    rng = np.random.default_rng(9)
    g = np.concatenate(vs + ([(rng.standard_normal(filler) * 1e-3).astype(np.float32)] if filler else []))
    d = g.size
    x0 = np.zeros(d, dtype=np.float32)
    orc = so.Oracle(1, sizes, x0, compressor=so.SIGN, avg_period=0, momentum=0.0)
    gpu = sb.Sae(1, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=0, momentum=0.0)
    orc.step(g.reshape(1, d), 1.0)
    gpu.step(torch.from_numpy(g).cuda().view(1, d), 1.0)
    gpu.sync()
    got = gpu.get_state(sb.STATE_WORKER_SCALES, 0).cpu().numpy()
    exp = orc.get(orc.SCALES, 0)
    for j, v in enumerate(vs):
        S = scale_cases.fixed_sum(v)
        t, r = scale_cases.scale_truncating(S, v.size), scale_cases.scale_rounding(S, v.size)
        assert t != r
        assert exp[j] == t, (j, exp[j], t, r)
        assert got[j] == t, (j, got[j], t, r)
    assert np.array_equal(got.view(np.uint32), exp.view(np.uint32))
    # the server compresses e + C(v) = +-s: its scale is s again, and the whole state follows the oracle
    assert np.array_equal(gpu.get_state(sb.STATE_SERVER_SCALES).cpu().numpy().view(np.uint32),
                          orc.get(orc.SCALES_SRV).view(np.uint32))
    assert np.array_equal(gpu.get_params().cpu().numpy().view(np.uint32), orc.get(orc.X).view(np.uint32))
    gpu.close()


@pytest.mark.parametrize("K,p", [(4, 1), (8, 1), (2, 0)])
def test_discriminating_sums_inside_a_multi_worker_step(K, p):
    """The same tensors as the first gradients of K workers (worker k gets them scaled by 2^-k: still
    discriminating, a power-of-two scaling shifts the sum), then two ordinary steps: the folded p = 1 worker
    pass and the unfolded one read the scales these sums produced."""
    import torch
    vs = _tensors(11)
    sizes = [v.size for v in vs]
    base = np.concatenate(vs)
    d = base.size
    rng = np.random.default_rng(K)
    x0 = (rng.standard_normal(d) * 0.05).astype(np.float32)
    orc = so.Oracle(K, sizes, x0, compressor=so.SIGN, avg_period=p, momentum=0.0)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=p, momentum=0.0)
    g0 = np.stack([base * np.float32(2.0 ** -k) for k in range(K)])
    for t in range(3):
        g = g0 if t == 0 else (rng.standard_normal((K, d)) * 1e-3).astype(np.float32)
        orc.step(g, 1.0)
        gpu.step(torch.from_numpy(g).cuda(), 1.0)
        gpu.sync()
        for k in range(K):
            got = gpu.get_state(sb.STATE_WORKER_SCALES, k).cpu().numpy()
            assert np.array_equal(got.view(np.uint32), orc.get(orc.SCALES, k).view(np.uint32)), (t, k)
            if t == 0:
                for j, v in enumerate(vs):
                    S = scale_cases.fixed_sum(g0[k][sum(sizes[:j]):sum(sizes[:j + 1])])
                    assert got[j] == scale_cases.scale_truncating(S, v.size) != scale_cases.scale_rounding(S, v.size)
        assert np.array_equal(gpu.get_params().cpu().numpy().view(np.uint32), orc.get(orc.X).view(np.uint32))
    gpu.close()
