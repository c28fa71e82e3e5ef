"""Checkpoint / resume and the gradient-mismatch diagnostics, against the oracle."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from parity_util import compare_state, compare_server_messages

pytestmark = pytest.mark.gpu

SIZES = [33, 4096, 5000, 700, 3 * 4096]


@pytest.mark.parametrize("mu", [0.9, 0.0])
@pytest.mark.parametrize("comp,p,K", [(so.SIGN, 1, 4), (so.SIGN, 3, 3), (so.TOPK, 2, 4), (so.TOPK, 1, 3), (so.SIGN, 0, 2)])
def test_resume_continues_bit_for_bit(comp, p, K, mu):
    """Save after 5 steps, restore into a fresh handle (different x0), continue: same bits as the oracle."""
    import torch
    d = sum(SIZES)
    scales = synth.tensor_scales(7, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(7, d)
    kw = dict(compressor=comp, avg_period=p, momentum=mu, weight_decay=1e-4, topk_num=1, topk_den=20)
    orc = so.Oracle(K, SIZES, x0, threads=4, **kw)
    a = sb.Sae(K, SIZES, torch.from_numpy(x0).cuda(), **kw)
    lrs = [0.1, 0.1, 0.05, 0.1, 0.2, 0.1, 0.05, 0.1, 0.1]
    for t in range(5):
        g = synth.grads_numpy(7, t, K, SIZES, scales)
        orc.step(g, lrs[t])
        a.step(torch.from_numpy(g).cuda(), lrs[t])
    blob = a.save_state()
    a.close()
    b = sb.Sae(K, SIZES, torch.zeros(d, device="cuda"), **kw)
    b.load_state(blob)
    assert b.iteration == 5
    compare_state(b, orc, comp, tag="restored")
    for t in range(5, 9):
        g = synth.grads_numpy(7, t, K, SIZES, scales)
        orc.step(g, lrs[t])
        b.step(torch.from_numpy(g).cuda(), lrs[t])
        compare_state(b, orc, comp, tag=f"resumed t={t + 1}")
        compare_server_messages(b, orc, comp, 1, tag=f"resumed t={t + 1}")
    # a checkpoint of another configuration is refused
    c = sb.Sae(K, SIZES, torch.zeros(d, device="cuda"), **dict(kw, momentum=0.5))
    with pytest.raises(sb.SaeError):
        c.load_state(blob)
    with pytest.raises(sb.SaeError):
        sb._check(sb.lib().sae_save_state(c.h, blob.data_ptr(), 16), "sae_save_state", c.h)


@pytest.mark.parametrize("comp,p", [(so.SIGN, 0), (so.SIGN, 1), (so.SIGN, 3), (so.TOPK, 2), (so.TOPK, 1)])
def test_gradient_mismatch_bounds(comp, p):
    """|| e + ebar ||^2 and (1/K) sum_k || e + ebar - e^(k) ||^2 (Section 3) from the oracle's errors."""
    import torch
    K = 4
    d = sum(SIZES)
    scales = synth.tensor_scales(8, len(SIZES), -4.0, -1.0)
    x0 = synth.x0_numpy(8, d)
    kw = dict(compressor=comp, avg_period=p, momentum=0.9, topk_num=1, topk_den=20)
    orc = so.Oracle(K, SIZES, x0, threads=4, **kw)
    gpu = sb.Sae(K, SIZES, torch.from_numpy(x0).cuda(), **kw)
    assert gpu.get_mismatch() == (0.0, 0.0)
    for t in range(6):
        g = synth.grads_numpy(8, t, K, SIZES, scales)
        orc.step(g, 0.1)
        gpu.step(torch.from_numpy(g).cuda(), 0.1)
        e = orc.get_all(orc.E).astype(np.float64)
        base = orc.get(orc.E_SRV).astype(np.float64) + e.mean(axis=0)
        exp_ef = float((base ** 2).sum())
        exp_saef = float((((base[None, :] - e) ** 2).sum(axis=1)).mean())
        got_ef, got_saef = gpu.get_mismatch()
        assert got_ef == pytest.approx(exp_ef, rel=1e-9, abs=1e-30)
        assert got_saef == pytest.approx(exp_saef, rel=1e-9, abs=1e-30)
        if p > 0 and (orc.iteration + 1) % p == 0:
            # right after error averaging every e^(k) equals ebar: the step-ahead bound is || e ||^2
            assert got_saef == pytest.approx(float((orc.get(orc.E_SRV).astype(np.float64) ** 2).sum()), rel=1e-9, abs=1e-30)
