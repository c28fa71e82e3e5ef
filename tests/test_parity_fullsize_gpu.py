"""Full-size parity (configs 2, 3, 4) in the launch configuration the benchmark times.  Every tensor is
an independent problem (compression is per tensor, everything else per element), so the oracle
reproduces a sample of whole tensors -- the largest, ragged ones, small ones -- over the trajectory
from the same seeded gradients, and the GPU results for those tensors must match bit for bit."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import configs, synth
from parity_util import assert_same

pytestmark = pytest.mark.gpu


def sample_tensors(sizes, budget):
    order = np.argsort(sizes)
    fits = [int(j) for j in order[::-1] if sizes[j] <= budget]
    pick = fits[:1] + [int(order[0]), int(order[len(order) // 2]), len(sizes) - 1, len(sizes) - 2]
    rng = np.random.default_rng(0)
    pick += [int(j) for j in rng.permutation(len(sizes))[:12]]
    out, total = [], 0
    for j in dict.fromkeys(pick):
        if total + sizes[j] <= budget or not out:
            out.append(j)
            total += sizes[j]
    return sorted(out)


def run_fullsize(idx, p, steps, budget, seed=0):
    """Runs on a non-default stream, as bench.py does: the steps are captured and replayed as CUDA graphs."""
    import torch
    with torch.cuda.stream(torch.cuda.Stream()):
        _run_fullsize(idx, p, steps, budget, seed)
    torch.cuda.synchronize()


def _run_fullsize(idx, p, steps, budget, seed):
    import psutil
    import torch
    w = configs.workload(idx)
    K, sizes, d = w.num_workers, w.tensor_sizes, w.d
    # the oracle holds ~6 K x n float arrays for the sampled tensors: stay far inside the host's memory
    budget = int(min(budget, psutil.virtual_memory().available // (K * 4 * 24)))
    offs = np.concatenate([[0], np.cumsum(sizes)])
    scales = synth.workload_scales(w, seed)
    gen = synth.DeviceGenerator(sizes, scales)
    x0 = torch.empty(d, device="cuda")
    gen.x0(x0, seed)
    gpu = sb.Sae(K, sizes, x0, compressor=w.compressor, avg_period=p, momentum=w.momentum, weight_decay=w.weight_decay,
                 topk_num=w.topk_num, topk_den=w.topk_den)
    js = sample_tensors(sizes, budget)
    sub_sizes = [sizes[j] for j in js]
    x0_sub = np.concatenate([synth.x0_numpy_range(seed, int(offs[j]), sizes[j]) for j in js])
    orc = so.Oracle(K, sub_sizes, x0_sub, compressor=w.compressor, avg_period=p, momentum=w.momentum,
                    weight_decay=w.weight_decay, topk_num=w.topk_num, topk_den=w.topk_den, threads=so.max_threads())
    idx_sub = torch.from_numpy(np.concatenate([np.arange(offs[j], offs[j + 1]) for j in js])).cuda()
    gbuf = [torch.empty(K, d, device="cuda") for _ in range(2)]     # two buffers, as the bench's ring: graph keys repeat
    take = lambda t: t[idx_sub].cpu().numpy()
    check_at = set(range(3)) | set(range(steps - 1, 2, -max(1, steps // 4)))
    for t in range(steps):
        g = gbuf[t % 2]
        gen.grads(g, K, seed, t, w.outlier_per_65536, w.outlier_mult)
        gpu.step(g, w.lr)
        g_sub = g[:, idx_sub].cpu().numpy()
        if t == 0:
            # the device generator against the numpy one (afterwards the gathered device values feed the oracle)
            g_np = np.stack([np.concatenate([synth.grads_numpy_range(seed, t, k, int(offs[j]), sizes[j], scales[j],
                                                                     w.outlier_per_65536, w.outlier_mult) for j in js])
                             for k in range(K)])
            assert_same(f"cfg{idx} gradient sample t={t}", g_sub, g_np)
        orc.step(g_sub, w.lr)
        if t not in check_at:
            continue
        gpu.sync()
        tag = f"cfg{idx} p={p} t={t + 1}"
        assert_same(f"{tag} x", take(gpu.get_params()), orc.get(orc.X))
        assert_same(f"{tag} e_srv", take(gpu.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
        for k in sorted({0, K // 2, K - 1}):
            assert_same(f"{tag} m[{k}]", take(gpu.get_state(sb.STATE_MOMENTUM, k)), orc.get(orc.M, k))
            assert_same(f"{tag} e[{k}]", take(gpu.get_state(sb.STATE_WORKER_ERROR, k)), orc.get(orc.E, k))
            if w.compressor == configs.SIGN:
                sc = gpu.get_state(sb.STATE_WORKER_SCALES, k).cpu().numpy()[js]
                assert_same(f"{tag} scales[{k}]", sc, orc.get(orc.SCALES, k))
            else:
                ta = gpu.get_state(sb.STATE_WORKER_TAU, k).cpu().numpy().view(np.uint32)[js]
                assert_same(f"{tag} tau[{k}]", ta.astype(np.uint64), orc.tau(k))
    assert not orc.range_flag
    gpu.close()


@pytest.mark.parametrize("p,steps", [(1, 100), (20, 45)])
def test_config2_fullsize(p, steps):
    """p = 1: all 100 iterations of the workload; p = 20: two averaging events."""
    run_fullsize(2, p, steps, budget=4_000_000)


@pytest.mark.parametrize("p,steps", [(1, 100), (20, 45)])
def test_config3_fullsize(p, steps):
    run_fullsize(3, p, steps, budget=4_000_000)


@pytest.mark.parametrize("p,steps", [(1, 50), (2, 10)])
def test_config4_fullsize(p, steps):
    """32 workers x 109.5 M parameters: element offsets beyond 2^31, byte offsets beyond 2^32.
    p = 1 runs all 50 iterations with the folded-in averaging (from the second step on), p = 2 alternates
    stored and recomputed model differences."""
    run_fullsize(4, p, steps, budget=2_500_000)


def test_config4_embedding_scale_first_step():
    """The 23.4 M-element embedding spans 5723 tiles per worker.  At the first step Delta = fl(eta g)
    (m_0 = e_0 = 0), so its scale is the oracle's compressor applied to that one row."""
    import torch
    w = configs.workload(4)
    K, sizes, d = w.num_workers, w.tensor_sizes, w.d
    scales = synth.workload_scales(w, 0)
    gen = synth.DeviceGenerator(sizes, scales)
    x0 = torch.zeros(d, device="cuda")
    gpu = sb.Sae(K, sizes, x0, compressor=sb.SIGN, avg_period=1, momentum=w.momentum)
    g = torch.empty(K, d, device="cuda")
    gen.grads(g, K, 0, 0)
    gpu.step(g, w.lr)
    gpu.sync()
    n0 = sizes[0]
    for k in (0, K - 1):
        row = g[k, :n0].cpu().numpy()
        assert_same("embedding gradient", row, synth.grads_numpy_range(0, 0, k, 0, n0, scales[0]))
        delta = np.float32(w.lr) * row
        c, s, _, rg = so.compress(so.SIGN, delta)
        assert not rg
        got = gpu.get_state(sb.STATE_WORKER_SCALES, k).cpu().numpy()[0]
        assert_same(f"embedding scale[{k}]", np.array([got]), np.array([s], dtype=np.float32))
        words = gpu.get_state(sb.STATE_WORKER_WORDS, k).cpu().numpy().view(np.uint32)[: (n0 + 31) // 32]
        assert_same(f"embedding words[{k}]", words, so.pack_signs(delta, [n0]))
    gpu.close()


@pytest.mark.parametrize("p,steps", [(1, 8), (2, 6)])
def test_one_embedding_sized_tensor_whole_trajectory(p, steps):
    """The one shape a sample of whole tensors cannot reach at full worker count: a single tensor of
    23 440 896 elements (config 4's embedding) for 32 workers -- 5723 tiles per worker feeding one L1 record,
    the folded two-halves ring of the 32-worker pass on a tensor that never ends, the open server pass of the
    p = 1 form and (p = 2) stored and recomputed differences in turn.  Every step: parameters, server error,
    all 32 scales; first, middle and last step: every worker's momentum, error, step-ahead point and sign
    words, and the server's message."""
    import psutil
    import torch
    from parity_util import compare_state, compare_server_messages
    K, n = 32, 30522 * 768
    if psutil.virtual_memory().available < 6 * K * n * 4 + (8 << 30):
        pytest.skip("the oracle's arrays for this case need about 20 GB of host memory")
    sizes = [n]
    scales = synth.tensor_scales(4, 1, -5.0, -2.0)
    gen = synth.DeviceGenerator(sizes, scales)
    with torch.cuda.stream(torch.cuda.Stream()):
        x0 = torch.empty(n, device="cuda")
        gen.x0(x0, 4)
        kw = dict(compressor=so.SIGN, avg_period=p, momentum=0.9)
        gpu = sb.Sae(K, sizes, x0, **kw)
        orc = so.Oracle(K, sizes, x0.cpu().numpy(), threads=so.max_threads(), **kw)
        gbuf = [torch.empty(K, n, device="cuda") for _ in range(2)]
        for t in range(steps):
            g = gbuf[t % 2]
            gen.grads(g, K, 4, t)
            gpu.step(g, 0.1)
            gh = g.cpu().numpy()
            if t == 0:
                assert_same("generator row", gh[K - 1, -5000:],
                            synth.grads_numpy_range(4, 0, K - 1, n - 5000, 5000, scales[0]))
            orc.step(gh, 0.1)
            del gh
            tag = f"one tensor p={p} t={t + 1}"
            if t in (0, steps // 2, steps - 1):
                compare_state(gpu, orc, so.SIGN, tag=tag)
                compare_server_messages(gpu, orc, so.SIGN, 1, tag=tag)
            else:
                gpu.sync()
                assert_same(f"{tag} x", gpu.get_params().cpu().numpy(), orc.get(orc.X))
                assert_same(f"{tag} e_srv", gpu.get_state(sb.STATE_SERVER_ERROR).cpu().numpy(), orc.get(orc.E_SRV))
                for k in range(K):
                    assert_same(f"{tag} scale[{k}]", gpu.get_state(sb.STATE_WORKER_SCALES, k).cpu().numpy(),
                                orc.get(orc.SCALES, k))
        assert not orc.range_flag
        gpu.close()
