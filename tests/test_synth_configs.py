"""Host logic: workload parameter lists and the seeded input generator (numpy side)."""
import numpy as np
import pytest

from paper_2008_05823_b200 import configs, synth


def test_workload_totals():
    exp = {0: (4, 59, 269722, 8437), 1: (8, 167, 858868, 26860), 2: (16, 161, 25557032, 798658),
           3: (8, 161, 25557032, 798658), 4: (32, 199, 109482240, 3421320)}
    for i, (K, T, d, words) in exp.items():
        w = configs.workload(i)
        assert (w.num_workers, w.num_tensors, w.d) == (K, T, d)
        assert sum((n + 31) // 32 for n in w.tensor_sizes) == words
    assert min(configs.workload(2).tensor_sizes) == 64 and max(configs.workload(2).tensor_sizes) == 2359296
    assert max(configs.workload(4).tensor_sizes) == 30522 * 768
    with pytest.raises(ValueError):
        configs.workload(5)


def test_mix64_matches_between_int_and_numpy():
    zs = [0, 1, 2 ** 63, 2 ** 64 - 1, 0x123456789ABCDEF]
    with np.errstate(over="ignore"):
        got = synth._mix64_np(np.array(zs, dtype=np.uint64))
    assert [int(g) for g in got] == [synth.mix64_int(z) for z in zs]


def test_gradient_statistics_and_determinism():
    sizes = [1000, 50000, 7]
    scales = synth.tensor_scales(0, 3, -4.0, -1.0)
    assert np.all((scales >= 1e-4) & (scales <= 1e-1))
    g = synth.grads_numpy(0, 3, 2, sizes, scales)
    g2 = synth.grads_numpy(0, 3, 2, sizes, scales, chunk=977)
    np.testing.assert_array_equal(g, g2)                      # chunking does not change values
    assert g.shape == (2, sum(sizes)) and g.dtype == np.float32
    z = g[:, 1000:51000] / scales[1]
    assert abs(z.mean()) < 0.02 and abs(z.std() - 1.0) < 0.02
    assert np.abs(z).max() < 6.0                              # Irwin-Hall of 12 is bounded by 6
    assert not np.array_equal(g[0], g[1])                     # workers are independent draws
    assert not np.array_equal(g, synth.grads_numpy(0, 4, 2, sizes, scales))
    assert not np.array_equal(g, synth.grads_numpy(1, 3, 2, sizes, scales))


def test_outliers():
    sizes = [200000]
    scales = np.array([1e-2], dtype=np.float32)
    g = synth.grads_numpy(5, 0, 1, sizes, scales)
    go = synth.grads_numpy(5, 0, 1, sizes, scales, outlier_per_65536=655, outlier_mult=50.0)
    changed = go != g
    frac = changed.mean()
    assert 0.008 < frac < 0.012
    np.testing.assert_array_equal(go[changed], g[changed] * np.float32(50.0))


def test_x0():
    x = synth.x0_numpy(0, 100000)
    assert abs(x.std() - 0.05) < 0.002 and abs(x.mean()) < 0.001
    np.testing.assert_array_equal(x[:1000], synth.x0_numpy(0, 1000))


def test_blockwise_sizes():
    from paper_2008_05823_b200 import configs
    assert configs.blockwise_sizes([10, 4, 3], 4) == [4, 4, 2, 4, 3]
    assert configs.blockwise_sizes([8], 4) == [4, 4]
    sizes = configs.resnet50_sizes()
    blk = configs.blockwise_sizes(sizes, 4096)
    assert sum(blk) == sum(sizes) and max(blk) == 4096
    assert len(blk) == sum((n + 4095) // 4096 for n in sizes)
    import pytest
    with pytest.raises(ValueError):
        configs.blockwise_sizes([8], 0)
