"""Large problems (K * d > 2^24: the persistent worker passes with their folded tails, the deferred server lines,
graph replay on a side stream) with seeded random calls between the steps -- getters, diagnostics, a checkpoint
taken and restored, profiling switched on and off.  None of these may change a bit of the trajectory, and each
getter must return the oracle's value at the moment it is called, whatever part of a step was still open."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from parity_util import compare_state, compare_server_messages, assert_same

pytestmark = pytest.mark.gpu

OPS = ["none"] * 8 + ["params", "step_ahead", "server_error", "worker_error", "worker_message",
       "server_message", "mismatch", "checkpoint", "profiling", "sync", "momentum"]      # half of the gaps stay empty


# the folded forms by name, so that the draw cannot miss them: (K, compressor, p) with momentum and no weight decay
FORCED = [(8, so.TOPK, 1), (16, so.TOPK, 1), (16, so.TOPK, 0), (32, so.SIGN, 1), (16, so.SIGN, 1), (32, so.SIGN, 1)]
NUM_DRAWN = 24


def draw(case):
    rng = np.random.default_rng(7000 + case)
    forced = FORCED[case - NUM_DRAWN] if case >= NUM_DRAWN else None
    K = forced[0] if forced else int(rng.choice([8, 16, 32]))
    big = (1 << 24) // K + int(rng.integers(1, 50_000))           # one tensor that alone crosses the limit
    sizes = [int(s) for s in rng.choice([1, 33, 4096, 5000, 70_000], size=int(rng.integers(1, 4)))]
    sizes.insert(int(rng.integers(0, len(sizes) + 1)), big)
    comp, p = int(rng.choice([so.SIGN, so.TOPK])), int(rng.choice([1, 1, 0, 3]))
    mu, lam = float(rng.choice([0.9, 0.9, 0.0])), float(rng.choice([0.0, 0.0, 0.0, 1e-4]))
    if forced:
        comp, p, mu, lam = forced[1], forced[2], 0.9, 0.0
    return dict(K=K, sizes=sizes, comp=comp, p=p, mu=mu, lam=lam,
                dc=int(rng.integers(0, 2)),
                side_stream=bool(rng.integers(0, 2)),
                ops=[str(o) for o in rng.choice(OPS, size=9)],
                lrs=[float(x) for x in rng.choice([0.05, 0.1, 0.2], size=2)],
                seed=int(rng.integers(0, 1 << 20)))


def apply_op(op, gpu, orc, c, tag):
    cpu = lambda t: t.cpu().numpy()
    K = c["K"]
    k = orc.iteration % K
    if op == "params":
        assert_same(f"{tag} x", cpu(gpu.get_params()), orc.get(orc.X))
    elif op == "step_ahead":
        assert_same(f"{tag} step_ahead[{k}]", cpu(gpu.get_step_ahead(k)), orc.step_ahead(k))
    elif op == "server_error":
        assert_same(f"{tag} e_srv", cpu(gpu.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
    elif op == "worker_error":
        assert_same(f"{tag} e[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_ERROR, k)), orc.get(orc.E, k))
    elif op == "momentum" and gpu.keeps_momentum:
        assert_same(f"{tag} m[{k}]", cpu(gpu.get_state(sb.STATE_MOMENTUM, k)), orc.get(orc.M, k))
    elif op == "worker_message":
        if c["comp"] == so.SIGN:
            assert_same(f"{tag} scales[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_SCALES, k)), orc.get(orc.SCALES, k))
            assert_same(f"{tag} words[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_WORDS, k)).view(np.uint32),
                        so.pack_signs(orc.get(orc.DELTA, k), orc.sizes))
        else:
            assert_same(f"{tag} tau[{k}]",
                        cpu(gpu.get_state(sb.STATE_WORKER_TAU, k)).view(np.uint32).astype(np.uint64), orc.tau(k))
    elif op == "server_message":
        compare_server_messages(gpu, orc, c["comp"], c["dc"], tag=tag)
    elif op == "mismatch":
        # || e + ebar ||^2 and (1/K) sum_k || e + ebar - e^(k) ||^2 (Section 3), from the oracle's errors in fp64
        e = orc.get_all(orc.E).astype(np.float64)
        base = orc.get(orc.E_SRV).astype(np.float64) + e.mean(axis=0)
        exp = (float((base ** 2).sum()), float((((base[None, :] - e) ** 2).sum(axis=1)).mean()))
        np.testing.assert_allclose(gpu.get_mismatch(), exp, rtol=1e-9, atol=1e-30, err_msg=tag)
    elif op == "checkpoint":
        blob = gpu.save_state()
        gpu.load_state(blob)
    elif op == "profiling":
        gpu.set_profiling(True)
        gpu.get_kernel_times()
        gpu.set_profiling(False)
    elif op == "sync":
        gpu.sync()


@pytest.mark.parametrize("case", range(NUM_DRAWN + len(FORCED)))
def test_random_calls_between_steps(case):
    import torch
    c = draw(case)
    K, sizes = c["K"], c["sizes"]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(c["seed"], len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(c["seed"], d)
    kw = dict(compressor=c["comp"], server_compress=c["dc"], avg_period=c["p"], momentum=c["mu"],
              weight_decay=c["lam"], topk_num=1, topk_den=100)
    orc = so.Oracle(K, sizes, x0, threads=8, **kw)
    stream = torch.cuda.Stream() if c["side_stream"] else torch.cuda.current_stream()
    with torch.cuda.stream(stream):
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
        pool = [synth.grads_numpy(c["seed"], t, K, sizes, scales, 1000, 100.0) for t in range(2)]
        dev = [torch.from_numpy(g).cuda() for g in pool]
        for t, op in enumerate(c["ops"]):
            lr = c["lrs"][(t // 3) % 2]
            orc.step(pool[t % 2], lr)
            gpu.step(dev[t % 2], lr)
            apply_op(op, gpu, orc, c, tag=f"case {case} {c} after step {t + 1}: {op}")
        compare_state(gpu, orc, c["comp"], tag=f"case {case} {c} end")
        compare_server_messages(gpu, orc, c["comp"], c["dc"], tag=f"case {case} end")
        assert not orc.range_flag
        gpu.close()


def test_two_handles_alternate_on_one_stream():
    """Two independent problems in the folded Top-K form stepped in turn on the same side stream: each handle
    forks part of its step onto a stream of its own and joins it again, so neither may disturb the other."""
    import torch
    cases = [draw(NUM_DRAWN + 0), draw(NUM_DRAWN + 1)]            # K = 8 and K = 16, Top-K, p = 1
    with torch.cuda.stream(torch.cuda.Stream()):
        runs = []
        for c in cases:
            K, sizes = c["K"], c["sizes"]
            d = int(np.sum(sizes))
            scales = synth.tensor_scales(c["seed"], len(sizes), -4.0, -1.0)
            x0 = synth.x0_numpy(c["seed"], d)
            kw = dict(compressor=c["comp"], server_compress=1, avg_period=c["p"], momentum=0.9, topk_num=1, topk_den=100)
            pool = [synth.grads_numpy(c["seed"], t, K, sizes, scales, 1000, 100.0) for t in range(2)]
            runs.append(dict(orc=so.Oracle(K, sizes, x0, threads=8, **kw),
                             gpu=sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw),
                             pool=pool, dev=[torch.from_numpy(g).cuda() for g in pool]))
        for t in range(6):
            for r in runs:
                r["orc"].step(r["pool"][t % 2], 0.1)
                r["gpu"].step(r["dev"][t % 2], 0.1)
        for i, r in enumerate(runs):
            compare_state(r["gpu"], r["orc"], so.TOPK, tag=f"handle {i}")
            compare_server_messages(r["gpu"], r["orc"], so.TOPK, 1, tag=f"handle {i}")
            r["gpu"].close()
