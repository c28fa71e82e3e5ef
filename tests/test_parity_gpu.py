"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs,
element by element, after every step.  Sign words, Top-K thresholds and index sets must be bit-exact;
floats are held to the stated 1e-5 relative bar (and are expected to be bit-identical)."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import configs, synth
from parity_util import compare_state, compare_server_messages, assert_same

pytestmark = pytest.mark.gpu

RAGGED = [1, 2, 31, 32, 33, 1000, 4097, 4096, 5000, 8192 + 5, 3 * 4096]


def run_pair(K, sizes, comp, steps, seed=0, p=0, dc=1, mode=so.SAEF, mu=0.9, lam=0.0, num=1, den=100, lrs=None,
             scale=1e-2, outliers=(0, 1.0), every=1):
    import torch
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(seed, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(seed, d)
    orc = so.Oracle(K, sizes, x0, compressor=comp, server_compress=dc, mode=mode, avg_period=p, momentum=mu,
                    weight_decay=lam, topk_num=num, topk_den=den, threads=4)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=comp, server_compress=dc, mode=mode, avg_period=p,
                 momentum=mu, weight_decay=lam, topk_num=num, topk_den=den)
    compare_state(gpu, orc, comp, tag="t=0")
    for t in range(steps):
        g = synth.grads_numpy(seed, t, K, sizes, scales, outliers[0], outliers[1])
        lr = 0.1 if lrs is None else lrs[t % len(lrs)]
        orc.step(g, lr)
        gpu.step(torch.from_numpy(g).cuda(), lr)
        if (t + 1) % every == 0 or t == steps - 1:
            tag = f"K={K} comp={comp} p={p} dc={dc} mode={mode} t={t + 1}"
            compare_state(gpu, orc, comp, tag=tag)
            compare_server_messages(gpu, orc, comp, dc, tag=tag)
    assert not orc.range_flag
    gpu.close()


@pytest.mark.parametrize("K", [1, 2, 3, 4])
@pytest.mark.parametrize("p", [0, 1, 3])
def test_sign_ragged(K, p):
    run_pair(K, RAGGED, so.SIGN, 7, p=p, lrs=[0.1, 0.05, 0.2])


@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("mode", [so.EF, so.SAEF])
@pytest.mark.parametrize("mu,lam", [(0.0, 0.0), (0.9, 1e-4), (0.5, 1e-2)])
def test_sign_variants(dc, mode, mu, lam):
    run_pair(3, RAGGED, so.SIGN, 6, p=2, dc=dc, mode=mode, mu=mu, lam=lam, seed=1)


@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("p", [0, 1, 3])
def test_sign_weight_decay_small_problem_without_getters_in_between(dc, p):
    """Weight decay makes the worker lines read x, so the server lines of a step cannot wait for the next server
    pass; on small problems the next worker pass carries them out itself.  State compared every fourth step only,
    so that most steps find the previous one's lines still pending; a steady p = 1 step is then two launches."""
    import torch
    K, sizes, seed = 3, RAGGED, 5
    run_pair(K, sizes, so.SIGN, 13, seed=seed, p=p, dc=dc, lam=5e-4, lrs=[0.1, 0.1, 0.05], every=4)
    if p == 1:
        d = int(np.sum(sizes))
        scales = synth.tensor_scales(seed, len(sizes), -4.0, -1.0)
        gpu = sb.Sae(K, sizes, torch.from_numpy(synth.x0_numpy(seed, d)).cuda(), compressor=so.SIGN, server_compress=dc,
                     avg_period=1, weight_decay=5e-4)
        g = torch.from_numpy(synth.grads_numpy(seed, 0, K, sizes, scales)).cuda()
        counts = []
        for t in range(6):
            gpu.step(g, 0.1)
            counts.append(gpu.kernel_launches)
        assert np.diff(np.array(counts))[-3:].tolist() == [2, 2, 2]
        gpu.close()


@pytest.mark.parametrize("K", [1, 3, 4])
@pytest.mark.parametrize("p", [0, 1, 3])
@pytest.mark.parametrize("num,den", [(1, 100), (1, 10)])
def test_topk_ragged(K, p, num, den):
    run_pair(K, RAGGED, so.TOPK, 6, p=p, num=num, den=den, outliers=(66, 100.0), seed=2)


@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("mode", [so.EF, so.SAEF])
def test_topk_variants(dc, mode):
    run_pair(2, RAGGED, so.TOPK, 5, p=2, dc=dc, mode=mode, mu=0.9, lam=1e-3, num=1, den=20, seed=1)


@pytest.mark.parametrize("K", [1, 3])
def test_identity(K):
    run_pair(K, RAGGED, so.IDENTITY, 5, p=2, lam=1e-3)


@pytest.mark.parametrize("K", [5, 40, 64])
def test_worker_counts_outside_the_folded_path(K):
    """K not a power of two, or above 32: p = 1 runs the plain worker pass and averages in the apply kernel."""
    run_pair(K, [33, 4096, 5000, 700], so.SIGN, 4, p=1, seed=4)
    run_pair(K, [33, 4096, 5000, 700], so.TOPK, 3, p=1, num=1, den=20, seed=4)


def test_single_large_ragged_tensor():
    """One tensor over many tiles whose size is not a multiple of 4 (ragged last row, odd gradient rows)."""
    run_pair(2, [9 * 4096 + 1235], so.SIGN, 5, p=1)
    run_pair(4, [9 * 4096 + 1235], so.SIGN, 5, p=2)
    run_pair(2, [9 * 4096 + 1235], so.TOPK, 5, p=2, num=1, den=50)


def test_topk_keep_everything():
    """num = den: k = n, Top-K is the identity except that exact zeros are never 'selected'."""
    run_pair(2, [100, 4096, 5000], so.TOPK, 4, p=2, num=1, den=1)


def test_topk_large_ratios_on_large_tensors():
    """Half and a quarter of the entries kept: every candidate region is as large as its tensor."""
    run_pair(2, [100, 40_000, 300_000], so.TOPK, 4, p=1, num=1, den=2)
    run_pair(4, [5000, 70_000, 3 * 4096], so.TOPK, 4, p=3, num=1, den=4, lrs=[0.1, 0.3, 0.02])


def test_sign_aligned_rows_vector_path():
    """d a multiple of 4 and tensors of whole tiles: every tile takes the 128-bit path."""
    run_pair(4, [4096, 8192, 4096 * 5, 64, 2048], so.SIGN, 6, p=1)
    run_pair(4, [4096, 8192, 4096 * 5, 64, 2048], so.SIGN, 6, p=3)
    run_pair(4, [4096, 8192, 4096 * 5, 64, 2048], so.TOPK, 6, p=3)


def test_topk_candidate_window_is_used_and_exact():
    """Steady gradients: after the first steps the threshold of a step is found among the candidates
    collected around the previous one (no extra pass over the data); every step stays exact."""
    import torch
    K, sizes, steps = 4, [20000, 3 * 4096, 100000, 700], 12
    d = sum(sizes)
    scales = synth.tensor_scales(5, len(sizes), -3.0, -2.0)
    x0 = synth.x0_numpy(5, d)
    orc = so.Oracle(K, sizes, x0, compressor=so.TOPK, avg_period=4, momentum=0.9, topk_num=1, topk_den=100, threads=4)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.TOPK, avg_period=4, momentum=0.9, topk_num=1,
                 topk_den=100)
    for t in range(steps):
        g = synth.grads_numpy(5, t, K, sizes, scales, 66, 100.0)
        orc.step(g, 0.1)
        gpu.step(torch.from_numpy(g).cuda(), 0.1)
        compare_state(gpu, orc, so.TOPK, tag=f"window t={t + 1}")
        compare_server_messages(gpu, orc, so.TOPK, 1, tag=f"window t={t + 1}")
    fb = gpu.get_state(sb.STATE_TOPK_FALLBACKS).cpu().numpy()
    # the first step has no previous threshold to look around: every pair misses, except for tensors small enough
    # that their candidate region holds them whole (here the 700-element one), which never need a guess
    assert K * (len(sizes) - 1) <= fb[0] < K * len(sizes) * steps // 2, fb
    assert len(sizes) - 1 <= fb[1] < len(sizes) * steps // 2, fb


def test_topk_ties_and_zeros():
    """Gradients quantised to a few levels: many exact ties at the threshold and exact zeros."""
    import torch
    K, sizes = 2, [100, 4096, 5000]
    d = sum(sizes)
    rng = np.random.default_rng(7)
    x0 = np.zeros(d, dtype=np.float32)
    orc = so.Oracle(K, sizes, x0, compressor=so.TOPK, avg_period=2, momentum=0.5, topk_num=1, topk_den=10)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.TOPK, avg_period=2, momentum=0.5, topk_num=1,
                 topk_den=10)
    for t in range(5):
        g = (rng.integers(-3, 4, (K, d)) * 0.25).astype(np.float32)
        g[:, :50] = 0
        orc.step(g, 0.5)
        gpu.step(torch.from_numpy(g).cuda(), 0.5)
        compare_state(gpu, orc, so.TOPK, tag=f"ties t={t + 1}")
        compare_server_messages(gpu, orc, so.TOPK, 1, tag=f"ties t={t + 1}")


def test_all_zero_gradients_and_tiny_values():
    """Degenerate inputs: zero gradients (scale 0, sign(0) = +), values below the 2^-64 fixed-point unit."""
    import torch
    K, sizes = 2, [33, 4096]
    d = sum(sizes)
    x0 = np.ones(d, dtype=np.float32)
    for comp in (so.SIGN, so.TOPK):
        orc = so.Oracle(K, sizes, x0, compressor=comp, avg_period=1)
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=comp, avg_period=1)
        for t, val in enumerate([0.0, 1e-30, 1e-42, 3.0]):
            g = np.full((K, d), val, dtype=np.float32)
            g[1] = -g[1]
            orc.step(g, 0.1)
            gpu.step(torch.from_numpy(g).cuda(), 0.1)
            compare_state(gpu, orc, comp, tag=f"degenerate comp={comp} t={t + 1}")


def test_large_values_take_the_integer_part_path():
    import torch
    K, sizes = 2, [1000, 4096]
    d = sum(sizes)
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal(d).astype(np.float32)
    orc = so.Oracle(K, sizes, x0, compressor=so.SIGN, avg_period=0)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=0)
    for t in range(3):
        g = (rng.standard_normal((K, d)) * np.exp(rng.uniform(-10, 18, (K, d)))).astype(np.float32)
        orc.step(g, 0.5)
        gpu.step(torch.from_numpy(g).cuda(), 0.5)
        compare_state(gpu, orc, so.SIGN, tag=f"large t={t + 1}")


def test_range_error_is_reported_and_sticky_until_sync():
    import torch
    sizes = [64]
    x0 = torch.zeros(64, device="cuda")
    gpu = sb.Sae(1, sizes, x0, compressor=sb.SIGN)
    g = torch.zeros(1, 64, device="cuda")
    g[0, 5] = float("inf")
    gpu.step(g, 0.1)
    with pytest.raises(sb.SaeError) as ei:
        gpu.sync()
    assert ei.value.status == sb.ERR_RANGE
    gpu.sync()          # cleared


def test_invalid_arguments():
    import torch
    x0 = torch.zeros(10, device="cuda")
    with pytest.raises(sb.SaeError):
        sb.Sae(0, [10], x0)
    with pytest.raises(sb.SaeError):
        sb.Sae(1, [10], x0, momentum=1.0)
    with pytest.raises(sb.SaeError):
        sb.Sae(1, [10], x0, compressor=7)
    gpu = sb.Sae(1, [10], x0)
    with pytest.raises(sb.SaeError):
        gpu.step(torch.zeros(1, 10, device="cuda"), 0.0)
    with pytest.raises(sb.SaeError):
        gpu.get_step_ahead(3)
    with pytest.raises(sb.SaeError):
        gpu.get_state(sb.STATE_WORKER_TAU)          # not a Top-K run


def test_device_generator_matches_numpy():
    import torch
    for idx in (0, 1):
        w = configs.workload(idx)
        scales = synth.workload_scales(w, 0)
        gen = synth.DeviceGenerator(w.tensor_sizes, scales)
        out = torch.empty(w.num_workers, w.d, device="cuda")
        for t in (0, 3):
            gen.grads(out, w.num_workers, 0, t, w.outlier_per_65536, w.outlier_mult)
            assert_same(f"grads cfg{idx} t={t}", out.cpu().numpy(), synth.workload_grads_numpy(w, 0, t, scales))
        x = torch.empty(w.d, device="cuda")
        gen.x0(x, 0)
        assert_same("x0", x.cpu().numpy(), synth.x0_numpy(0, w.d))


def test_step_host_and_get_params_host_match_device_path():
    import torch
    K, sizes = 3, RAGGED
    d = sum(sizes)
    x0 = torch.from_numpy(synth.x0_numpy(0, d)).cuda()
    a = sb.Sae(K, sizes, x0, avg_period=2)
    b = sb.Sae(K, sizes, x0, avg_period=2)
    scales = synth.tensor_scales(0, len(sizes), -4.0, -1.0)
    pinned = torch.empty(K, d).pin_memory()
    out_host = torch.empty(d).pin_memory()
    for t in range(4):
        g = synth.grads_numpy(0, t, K, sizes, scales)
        pinned.copy_(torch.from_numpy(g))
        a.step(torch.from_numpy(g).cuda(), 0.1)
        b.step_host(pinned, 0.1)
        b.get_params_host(out_host)
        assert_same("host path x", out_host.numpy(), a.get_params().cpu().numpy())


@pytest.mark.parametrize("comp,p", [(so.SIGN, 1), (so.SIGN, 3), (so.TOPK, 2)])
def test_graph_replay_on_a_side_stream(comp, p):
    """On a non-default stream a step is captured into a CUDA graph per (state, gradient pointer, lr)
    and replayed: cycle through two gradient buffers for many steps, compare with the oracle at the end
    and along the way."""
    import torch
    K, sizes = 4, RAGGED
    d = sum(sizes)
    scales = synth.tensor_scales(3, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(3, d)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        orc = so.Oracle(K, sizes, x0, compressor=comp, avg_period=p, weight_decay=1e-4, topk_den=20, threads=4)
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=comp, avg_period=p, weight_decay=1e-4, topk_den=20)
        gs = [synth.grads_numpy(3, t, K, sizes, scales) for t in range(2)]
        bufs = [torch.from_numpy(g).cuda() for g in gs]
        launches = []
        for t in range(14):
            orc.step(gs[t % 2], 0.1 if t < 10 else 0.05)
            gpu.step(bufs[t % 2], 0.1 if t < 10 else 0.05)
            launches.append(gpu.kernel_launches)
            if t in (5, 9, 13):
                compare_state(gpu, orc, comp, tag=f"graph comp={comp} p={p} t={t + 1}")
                compare_server_messages(gpu, orc, comp, 1, tag=f"graph comp={comp} p={p} t={t + 1}")
        per_step = np.diff(np.array(launches))
        assert per_step.min() >= 2          # replayed steps still account for their kernels (worker + server pass)
        gpu.close()


@pytest.mark.parametrize("comp,p", [(so.SIGN, 1), (so.TOPK, 0)])
def test_learning_rate_schedule_then_constant_on_a_side_stream(comp, p):
    """A learning rate that changes on every step (warm-up, then decay) for more steps than the graph cache
    tolerates misses, then held constant: steps run directly while it moves and as replayed graphs once it
    has settled -- the same bits as the oracle either way."""
    import torch
    K, sizes = 4, [33, 4096, 5000]
    d = sum(sizes)
    scales = synth.tensor_scales(5, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(5, d)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        orc = so.Oracle(K, sizes, x0, compressor=comp, avg_period=p, topk_den=20, threads=4)
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=comp, avg_period=p, topk_den=20)
        gs = [synth.grads_numpy(5, t, K, sizes, scales) for t in range(2)]
        bufs = [torch.from_numpy(g).cuda() for g in gs]
        lrs = [0.1 * (t + 1) / 40 for t in range(40)] + [0.1 * 0.97 ** t for t in range(40)] + [0.01] * 12
        for t, lr in enumerate(lrs):
            orc.step(gs[t % 2], lr)
            gpu.step(bufs[t % 2], lr)
            if t in (39, 79, 85, len(lrs) - 1):
                compare_state(gpu, orc, comp, tag=f"schedule comp={comp} t={t + 1}")
        gpu.close()


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
def test_two_runs_give_identical_bytes(comp):
    """Run-to-run determinism: the exact L1 is an integer sum (atomics in any order), histograms are integer
    counts, every float reduction has a fixed order -- two runs must agree byte for byte (zero signs included)."""
    import torch
    K, sizes = 4, RAGGED + [40000]
    d = sum(sizes)
    scales = synth.tensor_scales(9, len(sizes), -4.0, -1.0)
    x0 = torch.from_numpy(synth.x0_numpy(9, d)).cuda()
    gs = [torch.from_numpy(synth.grads_numpy(9, t, K, sizes, scales, 66, 100.0)).cuda() for t in range(6)]
    snaps = []
    for run in range(2):
        h = sb.Sae(K, sizes, x0, compressor=comp, avg_period=3, weight_decay=1e-4, topk_den=50)
        for g in gs:
            h.step(g, 0.1)
        h.sync()
        snaps.append(h.save_state().cpu().numpy().copy())
        h.close()
    assert np.array_equal(snaps[0], snaps[1])


def _trajectory(idx, p, steps, seed):
    w = configs.workload(idx)
    run_pair(w.num_workers, w.tensor_sizes, w.compressor, steps, seed=seed, p=p, mu=w.momentum, lam=w.weight_decay,
             num=w.topk_num, den=w.topk_den, lrs=[w.lr], outliers=(w.outlier_per_65536, w.outlier_mult),
             every=max(1, steps // 4))


def _trajectory_device_inputs(idx, p, steps, seed):
    """Whole trajectory of a workload with the gradients made by the device generator (itself checked against
    the numpy generator in test_device_generator_matches_numpy) and copied to the host for the oracle."""
    import torch
    w = configs.workload(idx)
    K, sizes, d = w.num_workers, w.tensor_sizes, w.d
    scales = synth.workload_scales(w, seed)
    gen = synth.DeviceGenerator(sizes, scales)
    x0 = torch.empty(d, device="cuda")
    gen.x0(x0, seed)
    kw = dict(compressor=w.compressor, avg_period=p, momentum=w.momentum, weight_decay=w.weight_decay,
              topk_num=w.topk_num, topk_den=w.topk_den)
    orc = so.Oracle(K, sizes, x0.cpu().numpy(), threads=so.max_threads(), **kw)
    gpu = sb.Sae(K, sizes, x0, **kw)
    g = torch.empty(K, d, device="cuda")
    for t in range(steps):
        gen.grads(g, K, seed, t, w.outlier_per_65536, w.outlier_mult)
        gpu.step(g, w.lr)
        orc.step(g.cpu().numpy(), w.lr)
        if (t + 1) % max(1, steps // 5) == 0 or t == steps - 1:
            compare_state(gpu, orc, w.compressor, tag=f"cfg{idx} p={p} t={t + 1}")
            compare_server_messages(gpu, orc, w.compressor, 1, tag=f"cfg{idx} p={p} t={t + 1}")
    assert not orc.range_flag
    gpu.close()


@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("p", [1, 5])
def test_config0_full_trajectory(seed, p):
    _trajectory(0, p, 10, seed)


@pytest.mark.parametrize("p", [1, 20])
def test_config1_full_trajectory(p):
    """All 200 iterations of config 1 (heavy-tailed gradients, weight decay)."""
    _trajectory_device_inputs(1, p, 200, 0)


@pytest.mark.parametrize("block,p", [(4096, 1), (4096, 0), (8192, 3), (1000, 1)])
def test_blockwise_sign(block, p):
    """Block-wise scaled sign (related work, Section 2): fixed-size segments of every tensor, each with its
    own scale; to the library a segment is a tensor of the list."""
    sizes = configs.blockwise_sizes([3 * 4096 + 17, 4096, 5, 20000, 8192], block)
    assert sum(sizes) == 3 * 4096 + 17 + 4096 + 5 + 20000 + 8192
    run_pair(4, sizes, so.SIGN, 6, p=p, lrs=[0.1, 0.05])


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK, so.IDENTITY])
@pytest.mark.parametrize("p,lam,mode", [(0, 0.0, so.SAEF), (3, 1e-4, so.SAEF), (2, 1e-4, so.EF), (1, 0.0, so.SAEF)])
def test_momentum_constant_zero(comp, p, lam, mode):
    """mu = 0 (the SGD / SignSGD variants of Section 5).  For p != 1 the library keeps no momentum rows at all
    (m^(k) is the step's gradient term); p = 1 goes through the regular paths.  Same bits either way."""
    run_pair(3, RAGGED, comp, 7, p=p, mu=0.0, lam=lam, mode=mode, num=1, den=20, outliers=(66, 100.0), seed=4,
             lrs=[0.1, 0.05])


def test_momentum_getter_is_refused_without_momentum_rows():
    import torch
    x0 = torch.zeros(sum(RAGGED), device="cuda")
    a = sb.Sae(2, RAGGED, x0, momentum=0.0, avg_period=0)
    assert not a.keeps_momentum
    with pytest.raises(sb.SaeError):
        a.get_state(sb.STATE_MOMENTUM, 0)
    a.get_state(sb.STATE_WORKER_ERROR, 0)
    a.close()
    b = sb.Sae(2, RAGGED, x0, momentum=0.0, avg_period=1)       # p = 1 keeps them (the folded averaging reads them)
    assert b.keeps_momentum
    b.get_state(sb.STATE_MOMENTUM, 0)
    b.close()


def test_maximum_worker_count():
    """K = 1024, the largest the library accepts (and 1025 is refused)."""
    import torch
    run_pair(1024, [33, 700], so.SIGN, 3, p=2, seed=5)
    run_pair(1024, [33, 700], so.TOPK, 2, p=0, num=1, den=10, seed=5)
    with pytest.raises(sb.SaeError):
        sb.Sae(1025, [33], torch.zeros(33, device="cuda"))


def test_maximum_tensor_size():
    """One tensor of 2^30 elements (the largest allowed: 262 144 tiles, the limit of the L1 record's headroom),
    one worker, single-way compression.  Too large for the CPU oracle to hold comfortably, so the step is
    checked against what Eq. 2 and Algorithm 1 fix for it: with K = 1, zero initial state and no server
    compression, Delta = lr * g, scale = mean |Delta| (within one fp32 rounding of the exactly rounded mean),
    bit i = (Delta_i >= 0), x_1 = x_0 - (+-scale), e^(1) = Delta - (+-scale)."""
    import torch
    n = 1 << 30
    gen = torch.Generator(device="cuda").manual_seed(7)
    g = torch.empty(1, n, device="cuda").normal_(0.0, 1e-2, generator=gen)
    x0 = torch.zeros(n, device="cuda")
    with pytest.raises(sb.SaeError):
        sb.Sae(1, [n + 1], torch.zeros(n + 1, device="cuda"))          # above the limit
    a = sb.Sae(1, [n], x0, compressor=sb.SIGN, server_compress=0, avg_period=0, momentum=0.9)
    a.step(g, 0.5)
    a.sync()
    delta = g[0] * 0.5                                                 # fma(0.5, m, 0) with m = fma(0.9, 0, g) = g: exact
    scale = a.get_state(sb.STATE_WORKER_SCALES, 0)
    exact = float(delta.double().abs().sum().item()) / n               # fp64 sum of 2^30 terms: ~1e-13 relative
    got = float(scale[0].item())
    assert abs(got - exact) <= 2.0 ** -23 * exact, (got, exact)
    words = a.get_state(sb.STATE_WORKER_WORDS, 0)
    pos = delta >= 0
    weights = (2 ** torch.arange(32, device="cuda", dtype=torch.int64))
    exp_words = (pos.view(-1, 32).to(torch.int64) * weights).sum(dim=1)
    assert torch.equal(words.to(torch.int64) & 0xFFFFFFFF, exp_words)
    del exp_words, weights
    code = torch.where(pos, scale[0], -scale[0])
    x1 = a.get_params()
    assert torch.equal(x1, x0 - code)
    del x1
    e1 = a.get_state(sb.STATE_WORKER_ERROR, 0)
    assert torch.equal(e1, delta - code)
    a.close()


@pytest.mark.parametrize("K", [8, 16, 32])
@pytest.mark.parametrize("lam", [0.0, 1e-4])
def test_folded_averaging_pass_ring_geometries(K, lam):
    """p = 1 with 8, 16 and 32 workers: the worker pass with the averaging folded in, in both of its ring
    geometries (3 deep stages up to 8 workers, 6 shallow ones from 16 on), on ragged and on whole tiles."""
    run_pair(K, [33, 4096, 5000, 700, 3 * 4096, 130], so.SIGN, 5, p=1, lam=lam, seed=6, lrs=[0.1, 0.05])


@pytest.mark.parametrize("comp", [so.SIGN, so.TOPK])
@pytest.mark.parametrize("K,p", [(2, 0), (3, 1), (4, 1), (4, 3), (16, 1), (5, 2)])
@pytest.mark.parametrize("dc", [0, 1])
def test_steps_without_getters_in_between(K, p, dc, comp):
    """With no getter between steps the server lines of a step are left pending and carried out inside the
    next step's server pass; the state is looked at only every fourth step here (and each look forces the
    pending lines), so both forms of the server pass and the switch between them are exercised."""
    run_pair(K, RAGGED, comp, 13, p=p, dc=dc, seed=8, lrs=[0.1, 0.05, 0.2], every=4, num=1, den=20,
             outliers=(66, 100.0))


def test_pending_server_lines_survive_a_checkpoint_and_a_side_stream():
    import torch
    d = int(np.sum(RAGGED))
    scales = synth.tensor_scales(9, len(RAGGED), -4.0, -1.0)
    x0 = synth.x0_numpy(9, d)
    kw = dict(compressor=so.SIGN, avg_period=3, momentum=0.9)
    orc = so.Oracle(4, RAGGED, x0, threads=4, **kw)
    with torch.cuda.stream(torch.cuda.Stream()):          # graph replay: the pending flag is part of the graph key
        a = sb.Sae(4, RAGGED, torch.from_numpy(x0).cuda(), **kw)
        gs = [torch.from_numpy(synth.grads_numpy(9, t, 4, RAGGED, scales)).cuda() for t in range(12)]
        for t in range(7):
            orc.step(gs[t].cpu().numpy(), 0.1)
            a.step(gs[t], 0.1)
        blob = a.save_state()                             # taken with a step's server lines pending
        b = sb.Sae(4, RAGGED, torch.zeros(d, device="cuda"), **kw)
        b.load_state(blob)
        for t in range(7, 12):
            orc.step(gs[t].cpu().numpy(), 0.1)
            a.step(gs[t], 0.1)
            b.step(gs[t], 0.1)
        compare_state(a, orc, so.SIGN, tag="continued")
        compare_state(b, orc, so.SIGN, tag="restored")
        compare_server_messages(a, orc, so.SIGN, 1, tag="continued")
        compare_server_messages(b, orc, so.SIGN, 1, tag="restored")
        a.close()
        b.close()
    torch.cuda.synchronize()


@pytest.mark.parametrize("K", [8, 16])
@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("every", [1, 2, 5])
@pytest.mark.parametrize("p", [1, 0, 3])
def test_topk_folded_tail(K, dc, every, p):
    """Top-K, K = 8 or 16, no weight decay: a step (with p != 1: one whose pre-step does not average) stops
    after its threshold select and the next step's worker pass does the rest; a getter in between carries
    the open tail out the unfolded way.  Looking at the state every step, every second step and every fifth
    step mixes both forms in every order."""
    run_pair(K, RAGGED + [40000], so.TOPK, 11, p=p, dc=dc, seed=11, lrs=[0.1, 0.05, 0.2], every=every, num=1, den=20,
             outliers=(66, 100.0))


@pytest.mark.parametrize("mode,mu", [(so.EF, 0.9), (so.SAEF, 0.5)])
def test_topk_folded_tail_branches(mode, mu):
    run_pair(8, RAGGED + [40000], so.TOPK, 9, p=0, mode=mode, mu=mu, seed=13, every=4, num=1, den=10, outliers=(66, 100.0))


@pytest.mark.parametrize("K", [8, 16])
@pytest.mark.parametrize("p", [1, 0, 4])
def test_topk_folded_tail_graph_replay_and_checkpoint(K, p):
    import torch
    sizes = RAGGED + [40000]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(12, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(12, d)
    kw = dict(compressor=so.TOPK, avg_period=p, momentum=0.9, topk_num=1, topk_den=20)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    with torch.cuda.stream(torch.cuda.Stream()):          # graph replay: the open tail is part of the graph key
        a = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
        gs = [torch.from_numpy(synth.grads_numpy(12, t, K, sizes, scales, 66, 100.0)).cuda() for t in range(4)]
        for t in range(9):
            orc.step(gs[t % 4].cpu().numpy(), 0.1)
            a.step(gs[t % 4], 0.1)
        blob = a.save_state()                             # taken with a tail open: the save closes it
        b = sb.Sae(K, sizes, torch.zeros(d, device="cuda"), **kw)
        b.load_state(blob)
        for t in range(9, 16):
            orc.step(gs[t % 4].cpu().numpy(), 0.1)
            a.step(gs[t % 4], 0.1)
            b.step(gs[t % 4], 0.1)
        compare_state(a, orc, so.TOPK, tag="continued")
        compare_state(b, orc, so.TOPK, tag="restored")
        compare_server_messages(a, orc, so.TOPK, 1, tag="continued")
        compare_server_messages(b, orc, so.TOPK, 1, tag="restored")
        a.close(); b.close()


@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("every", [1, 2, 3])
def test_sign_folded_server_pass(dc, every):
    """Scaled sign, p = 1, 32 workers, above the small-problem limit (K * d > 2^24), no weight decay: a step stops after its
    scales; the next step's worker pass adds the messages up in k order on the way and a streaming server pass
    reads that sum.  A getter in between runs the open server pass from the message words instead."""
    run_pair(32, [500_000, 33, 70_000, 4096], so.SIGN, 7, p=1, dc=dc, seed=14, lrs=[0.1, 0.05, 0.2], every=every)


def test_sign_folded_server_pass_checkpoint_and_graphs():
    import torch
    K, sizes = 32, [550_000, 33, 100_000]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(15, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(15, d)
    kw = dict(compressor=so.SIGN, avg_period=1, momentum=0.9)
    orc = so.Oracle(K, sizes, x0, threads=4, **kw)
    with torch.cuda.stream(torch.cuda.Stream()):
        a = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
        gs = [torch.from_numpy(synth.grads_numpy(15, t, K, sizes, scales)).cuda() for t in range(3)]
        for t in range(5):
            orc.step(gs[t % 3].cpu().numpy(), 0.1)
            a.step(gs[t % 3], 0.1)
        blob = a.save_state()                             # taken with a server pass open: the save closes it
        b = sb.Sae(K, sizes, torch.zeros(d, device="cuda"), **kw)
        b.load_state(blob)
        for t in range(5, 9):
            orc.step(gs[t % 3].cpu().numpy(), 0.1)
            a.step(gs[t % 3], 0.1)
            b.step(gs[t % 3], 0.1)
        compare_state(a, orc, so.SIGN, tag="continued")
        compare_state(b, orc, so.SIGN, tag="restored")
        compare_server_messages(a, orc, so.SIGN, 1, tag="continued")
        compare_server_messages(b, orc, so.SIGN, 1, tag="restored")
        a.close(); b.close()


@pytest.mark.parametrize("K,comp,dc,mode", [(32, so.SIGN, 1, so.SAEF), (16, so.SIGN, 1, so.SAEF), (4, so.SIGN, 0, so.SAEF),
                                            (8, so.SIGN, 1, so.EF), (8, so.TOPK, 1, so.SAEF), (16, so.TOPK, 0, so.SAEF)])
def test_step_ahead_point_read_after_every_step(K, comp, dc, mode):
    """Algorithm 1 as the paper runs it (p = 1): after every step the caller fetches the point where the next
    gradient is evaluated, x_{t+1} - e_{t+1}^(k).  Above the small-problem limit, on a side stream (step
    graphs), with unaligned output buffers; the caller also stops reading for a few steps and resumes, and
    reads the plain parameters in between.  Every fetched vector and, at the end, the whole state against
    the oracle."""
    import torch
    big = (1 << 24) // K + 40_000
    sizes = [33, 4096, big - 70_000, 5000, 3 * 4096 + 7, 60_000]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(21, len(sizes), -4.0, -1.0)
    x0 = synth.x0_numpy(21, d)
    kw = dict(compressor=comp, server_compress=dc, mode=mode, avg_period=1, momentum=0.9, topk_den=50)
    orc = so.Oracle(K, sizes, x0, threads=8, **kw)
    with torch.cuda.stream(torch.cuda.Stream()):
        gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
        gs = [synth.grads_numpy(21, t, K, sizes, scales) for t in range(2)]
        bufs = [torch.from_numpy(g).cuda() for g in gs]
        raw = torch.empty(d + 3, device="cuda")
        quiet = {5, 6, 7}                                   # steps after which nobody reads
        for t in range(12):
            lr = 0.1 if t < 9 else 0.05
            orc.step(gs[t % 2], lr)
            gpu.step(bufs[t % 2], lr)
            if t in quiet:
                continue
            out = raw[t % 4:t % 4 + d]                      # any 4-byte alignment
            w = t % K
            gpu.get_step_ahead(w, out)
            assert_same(f"step-ahead point t={t + 1} worker {w}", out.cpu().numpy(), orc.step_ahead(w))
            if t % 3 == 0:
                gpu.get_params(out)
                assert_same(f"x t={t + 1}", out.cpu().numpy(), orc.get(orc.X))
        compare_state(gpu, orc, comp, tag="read every step, end")
        compare_server_messages(gpu, orc, comp, dc, tag="read every step, end")
        gpu.close()


@pytest.mark.parametrize("K,p", [(8, 1), (8, 0), (2, 3), (16, 1)])
def test_topk_thresholds_that_jump(K, p):
    """Learning rates that jump by factors of 4 and 20: the thresholds leave their candidate windows in both
    directions -- upwards past the range the one-launch select bins finely (found among the list's keys above
    it), downwards out of the list altogether (the window fails: small tensors settled inside the block, large
    ones by the distributed select).  Tensors of every class: one that fits its candidate region whole, small and
    medium ones, and two whose regions are long enough for the wide blocks / the chunked lists.  Thresholds,
    selection masks and state against the oracle after every step."""
    import torch
    sizes = [700, 33, 5000, 40_000, 2_100_000 // K + 4096 * 3 + 5, 2_600_000 // K]
    d = int(np.sum(sizes))
    scales = synth.tensor_scales(31, len(sizes), -3.0, -2.0)
    x0 = synth.x0_numpy(31, d)
    kw = dict(compressor=so.TOPK, avg_period=p, momentum=0.9, topk_num=1, topk_den=10)
    orc = so.Oracle(K, sizes, x0, threads=8, **kw)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), **kw)
    lrs = [0.1] * 4 + [0.4] * 2 + [0.02] * 3 + [0.1] * 2 + [2.0, 0.001, 0.1]
    for t, lr in enumerate(lrs):
        g = synth.grads_numpy(31, t, K, sizes, scales, 66, 100.0)
        orc.step(g, lr)
        gpu.step(torch.from_numpy(g).cuda(), lr)
        tag = f"jump K={K} p={p} t={t + 1} lr={lr}"
        gpu.sync()
        for k in (0, K - 1):
            assert_same(f"{tag} tau[{k}]", gpu.get_state(sb.STATE_WORKER_TAU, k).cpu().numpy().view(np.uint32).astype(np.uint64),
                        orc.tau(k))
        assert_same(f"{tag} tau_srv", gpu.get_state(sb.STATE_SERVER_TAU).cpu().numpy().view(np.uint32).astype(np.uint64),
                    orc.tau(-1))
        if t % 3 == 2 or t == len(lrs) - 1:
            compare_state(gpu, orc, so.TOPK, tag=tag)
            compare_server_messages(gpu, orc, so.TOPK, 1, tag=tag)
    fb = gpu.get_state(sb.STATE_TOPK_FALLBACKS).cpu().numpy()
    assert fb[0] > K * (len(sizes) - 1)          # windows did fail after the first step as well
    gpu.close()
