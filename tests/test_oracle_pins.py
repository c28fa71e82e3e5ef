"""Pins for the CPU oracle: every check compares it with something other than itself -- a hand-worked
fixture, a closed form, an identity from the paper, a textbook routine written independently in numpy,
exact rational arithmetic, or brute force on tiny inputs."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import sae_oracle as so
import scale_cases
from oracle.sae_oracle import Oracle, IDENTITY, SIGN, TOPK, EF, SAEF

GOLD = os.path.join(os.path.dirname(__file__), "golden")
RNG = np.random.default_rng(1234)


def _lines(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


def rand_sizes_grads(K, sizes, steps, dtype, scale=1e-2, seed=0):
    rng = np.random.default_rng(seed)
    d = int(np.sum(sizes))
    x0 = rng.standard_normal(d).astype(dtype) * 0.05
    gs = [(rng.standard_normal((K, d)) * scale).astype(dtype) for _ in range(steps)]
    return x0, gs


# ------------------------------------------------------------------------------------------------
# compressors alone
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_scaled_sign_golden(dtype):
    """Eq. 2 on hand-worked vectors (tests/golden/scaled_sign_small.txt)."""
    for ln in _lines("scaled_sign_small.txt"):
        vec, scale = ln.split("|")
        v = np.array(vec.split(), dtype=dtype)
        s_exp = dtype(scale)
        c, s, _, rg = so.compress(SIGN, v)
        assert not rg
        assert s == s_exp
        exp = np.where(v >= 0, s_exp, -s_exp).astype(dtype)
        np.testing.assert_array_equal(c, exp)


def test_sign_words_golden():
    for ln in _lines("sign_words_small.txt"):
        sizes, vals, words = ln.split("|")
        sizes = [int(s) for s in sizes.split()]
        v = np.array(vals.split(), dtype=np.float32)
        exp = np.array([int(w, 16) for w in words.split()], dtype=np.uint32)
        np.testing.assert_array_equal(so.pack_signs(v, sizes), exp)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_topk_golden(dtype):
    for ln in _lines("topk_small.txt"):
        frac, vec, exp = ln.split("|")
        num, den = [int(a) for a in frac.split()]
        v = np.array(vec.split(), dtype=dtype)
        c, _, _, _ = so.compress(TOPK, v, num, den)
        np.testing.assert_array_equal(c, np.array(exp.split(), dtype=dtype))


def _exact_fixed_sum(v):
    """sum floor(|v| 2^64) with exact rationals."""
    return sum(int(Fraction(abs(float(a))) * (1 << 64)) for a in v)


def test_l1_fixed_matches_exact_rationals():
    for n, scale in [(1, 1.0), (7, 1e-3), (100, 1e-6), (1000, 3.0), (257, 1e-20), (64, 1e-38), (33, 1e5)]:
        v = (RNG.standard_normal(n) * scale).astype(np.float32)
        S, rg = so.l1_fixed(v)
        assert not rg
        assert S == _exact_fixed_sum(v)
    # values below 2^-64 contribute nothing; denormals included
    v = np.array([2.0 ** -65, 1e-45, -1e-40, 0.0, -0.0], dtype=np.float32)
    assert so.l1_fixed(v) == (0, False)
    # exactly 2^-64 is one unit; 1.0 is 2^64; 1.5 * 2^31 is exact
    assert so.l1_fixed(np.array([2.0 ** -64], dtype=np.float32))[0] == 1
    assert so.l1_fixed(np.array([-1.0], dtype=np.float32))[0] == 1 << 64
    assert so.l1_fixed(np.array([1.5 * 2.0 ** 31], dtype=np.float32))[0] == 3 << 94


def test_l1_fixed_permutation_invariant_and_range():
    v = (RNG.standard_normal(5000) * np.exp(RNG.uniform(-30, 5, 5000))).astype(np.float32)
    S0, _ = so.l1_fixed(v)
    for _ in range(3):
        assert so.l1_fixed(RNG.permutation(v))[0] == S0
    for bad in (np.inf, -np.inf, np.nan, 2.0 ** 32, -3e38):
        w = v.copy()
        w[17] = bad
        assert so.l1_fixed(w)[1] is True
    assert so.l1_fixed(np.array([np.nextafter(np.float32(2.0 ** 32), np.float32(0))], dtype=np.float32))[1] is False


def test_sign_scale_within_rounding_of_exact_mean():
    """The f32 scale is the exact mean of |v| up to: dropping < 2^-64 per element, truncation to 53
    bits, one double division, one rounding to float."""
    for n in (1, 3, 10, 1000, 4097):
        v = (RNG.standard_normal(n) * 1e-3).astype(np.float32)
        _, s, _, _ = so.compress(SIGN, v)
        exact = sum(Fraction(abs(float(a))) for a in v) / n
        assert abs(Fraction(float(s)) - exact) <= exact * Fraction(1, 2 ** 23)
        # the float-rounded exact value is at most one ulp away
        assert abs(float(s) - float(np.float32(float(exact)))) <= float(np.spacing(np.float32(float(exact))))


def test_scale_from_fixed_truncates_to_53_bits():
    """Eq. 2's ||v||_1 / n from the exact sum: the bits below the top 53 are dropped, not rounded in.
    S = 2^100 + 2^77 + 2^76 - 1, n = 1: float's last bit (2^77) is set, the next is clear and everything
    below is set.  Truncation leaves the quotient below the midpoint of two floats (-> 2^36 + 2^13);
    rounding the sum to 53 bits first would land on the midpoint and tie to even (-> 2^36 + 2^14)."""
    S = (1 << 100) + (1 << 77) + (1 << 76) - 1
    assert so.scale_from_fixed(S, 1) == np.float32(2.0 ** 36 + 2.0 ** 13)
    assert scale_cases.scale_truncating(S, 1) == np.float32(2.0 ** 36 + 2.0 ** 13)
    assert scale_cases.scale_rounding(S, 1) == np.float32(2.0 ** 36 + 2.0 ** 14)
    # bits below 2^48 of a 101-bit sum never matter
    assert so.scale_from_fixed((1 << 100) + (1 << 47) + 1, 1) == np.float32(2.0 ** 36)
    assert so.scale_from_fixed(0, 5) == 0.0


def test_scale_from_fixed_against_exact_rationals():
    """Random 60..120-bit sums and divisors against exact integer / fraction arithmetic written here."""
    rng = np.random.default_rng(77)
    for _ in range(4000):
        bits = int(rng.integers(1, 121))
        S = int(rng.integers(0, 1 << 62)) | (int(rng.integers(0, 1 << 62)) << 60)
        S = (S & ((1 << bits) - 1)) | (1 << (bits - 1))
        n = int(rng.integers(1, 1 << int(rng.integers(1, 31))))
        assert so.scale_from_fixed(S, n) == scale_cases.scale_truncating(S, n), (S, n)


@pytest.mark.parametrize("n", [1, 3, 8, 1000, 4097, 1 << 20])
@pytest.mark.parametrize("top_bit", [60, 75, 95])
def test_scale_from_fixed_where_truncating_and_rounding_differ(n, top_bit):
    """Sums built so that the two readings give different floats: the oracle follows the truncating one."""
    rng = np.random.default_rng(n + top_bit)
    for _ in range(5):
        S = scale_cases.discriminating_sum(n, top_bit, rng)
        t, r = scale_cases.scale_truncating(S, n), scale_cases.scale_rounding(S, n)
        assert t != r
        assert so.scale_from_fixed(S, n) == t


@pytest.mark.parametrize("n,top_bit", [(8, 60), (8, 90), (4096, 62), (5000, 70), (3 * 4096 + 7, 93)])
def test_sign_compress_on_tensors_where_truncating_and_rounding_differ(n, top_bit):
    """The same through the whole compressor: tensors whose exact L1 sum discriminates (values both below
    and above 1, mixed signs, zeros in between)."""
    v = scale_cases.discriminating_tensor(n, top_bit, seed=n)
    S = scale_cases.fixed_sum(v)
    assert so.l1_fixed(v) == (S, False)
    _, s, _, rg = so.compress(SIGN, v)
    assert not rg
    assert s == scale_cases.scale_truncating(S, n) != scale_cases.scale_rounding(S, n)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 1000, 4097])
def test_scaled_sign_closed_forms(n):
    """||v - C(v)||^2 = ||v||^2 - ||v||_1^2 / n, ||C(v)||_1 = ||v||_1, C(C(v)) = C(v)
    (so C is delta-approximate with delta = ||v||_1^2 / (n ||v||_2^2), Assumption 4)."""
    v = RNG.standard_normal(n)
    c, s, _, _ = so.compress(SIGN, v)
    l1, l2 = np.abs(v).sum(), (v * v).sum()
    assert np.isclose(((v - c) ** 2).sum(), l2 - l1 * l1 / n, rtol=1e-10, atol=1e-12)
    assert np.isclose(np.abs(c).sum(), l1, rtol=1e-12)
    c2, s2, _, _ = so.compress(SIGN, c)
    np.testing.assert_allclose(c2, c, rtol=1e-12)
    delta = l1 * l1 / (n * l2)
    assert ((v - c) ** 2).sum() <= (1 - delta) * l2 * (1 + 1e-10) + 1e-15
    # float32 instantiation: same facts to float rounding
    vf = v.astype(np.float32)
    cf, sf, _, _ = so.compress(SIGN, vf)
    assert np.isclose(float(sf), np.abs(vf.astype(np.float64)).mean(), rtol=3e-7)
    np.testing.assert_array_equal(np.signbit(cf), vf < 0)
    assert np.all(np.abs(cf) == sf)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_topk_bruteforce_tiny(dtype):
    """Full sort on tensors of <= 16 elements, with forced ties and zeros."""
    for trial in range(300):
        n = int(RNG.integers(1, 17))
        v = RNG.integers(-4, 5, n).astype(dtype) * dtype(0.25)      # many ties and zeros
        if trial % 3 == 0:
            v = RNG.standard_normal(n).astype(dtype)
        num, den = int(RNG.integers(1, 8)), 8
        kk = max(1, (n * num) // den)
        assert so.topk_count(n, num, den) == kk
        mags = np.sort(np.abs(v))[::-1]
        thr = mags[kk - 1]
        exp = np.where((np.abs(v) >= thr) & (v != 0), v, 0).astype(dtype)
        c, _, tau, _ = so.compress(TOPK, v, num, den)
        np.testing.assert_array_equal(c, exp)
        nz = np.count_nonzero(v)
        if len(np.unique(np.abs(v))) == n and nz == n:
            assert np.count_nonzero(c) == kk


def test_topk_contraction_and_full():
    for n, num, den in [(100, 1, 100), (1000, 1, 10), (1000, 1, 100), (37, 1, 2)]:
        v = RNG.standard_normal(n)
        c, _, _, _ = so.compress(TOPK, v, num, den)
        kk = max(1, n * num // den)
        assert ((v - c) ** 2).sum() <= (1 - kk / n) * (v * v).sum() + 1e-12
    v = RNG.standard_normal(50)
    np.testing.assert_array_equal(so.compress(TOPK, v, 1, 1)[0], v)
    np.testing.assert_array_equal(so.compress(IDENTITY, v)[0], v)


# ------------------------------------------------------------------------------------------------
# the iteration
# ------------------------------------------------------------------------------------------------
def momentum_sgd_numpy(x0, gs, K, mu, lr, wd=0.0):
    """Vanilla distributed momentum SGD (Section 2): x <- x - (eta/K) sum_k m_k, m_k <- mu m_k + g_k."""
    x = x0.astype(np.float64).copy()
    m = np.zeros((K, x.size))
    for g in gs:
        m = mu * m + g.astype(np.float64) + wd * x[None, :]
        x = x - lr * m.mean(axis=0)
    return x, m


@pytest.mark.parametrize("K", [1, 3, 4])
@pytest.mark.parametrize("mode", [EF, SAEF])
def test_identity_compressor_is_momentum_sgd(K, mode):
    sizes = [5, 1, 33, 100]
    x0, gs = rand_sizes_grads(K, sizes, 7, np.float64)
    o = Oracle(K, sizes, x0, compressor=IDENTITY, mode=mode, avg_period=2, momentum=0.9, weight_decay=1e-3,
               dtype=np.float64)
    for g in gs:
        o.step(g, 0.1)
    x_ref, m_ref = momentum_sgd_numpy(x0, gs, K, 0.9, 0.1, wd=1e-3)
    np.testing.assert_allclose(o.get(o.X), x_ref, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(o.get_all(o.M), m_ref, rtol=1e-12, atol=1e-14)
    assert np.all(o.get_all(o.E) == 0) and np.all(o.get(o.E_SRV) == 0)


@pytest.mark.parametrize("K", [1, 3])
@pytest.mark.parametrize("mode", [EF, SAEF])
@pytest.mark.parametrize("mu,lam", [(0.9, 1e-3), (0.0, 0.0), (0.5, 5e-2)])
def test_identity_compressor_matches_library_sgd(K, mode, mu, lam):
    """The same reduction against a library optimiser instead of a restatement: with the identity
    compressor the trajectory is torch.optim.SGD (heavy ball, no dampening, no Nesterov, weight decay
    added to the gradient) on the worker-averaged gradient, with a learning rate that changes per step."""
    import torch
    sizes = [7, 1, 40]
    x0, gs = rand_sizes_grads(K, sizes, 9, np.float64, seed=3)
    lrs = [0.1, 0.1, 0.05, 0.05, 0.2, 0.1, 0.01, 0.01, 0.1]
    o = Oracle(K, sizes, x0, compressor=IDENTITY, mode=mode, momentum=mu, weight_decay=lam, dtype=np.float64)
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=0.1, momentum=mu, weight_decay=lam)
    for g, lr in zip(gs, lrs):
        o.step(g, lr)
        for grp in opt.param_groups:
            grp["lr"] = lr
        p.grad = torch.tensor(g.astype(np.float64).mean(axis=0))
        opt.step()
    np.testing.assert_allclose(o.get(o.X), p.detach().numpy(), rtol=1e-11, atol=1e-13)


def test_identity_closed_form_constant_gradient():
    """K = 1, constant gradient: x_T = x_0 - eta g sum_{t=1..T} (1 - mu^t)/(1 - mu)."""
    sizes = [4, 3]
    d, T, mu, lr = 7, 12, 0.9, 0.05
    x0 = RNG.standard_normal(d)
    g = RNG.standard_normal((1, d))
    for comp in (IDENTITY,):
        o = Oracle(1, sizes, x0, compressor=comp, momentum=mu, dtype=np.float64)
        for _ in range(T):
            o.step(g, lr)
        coef = sum((1 - mu ** t) / (1 - mu) for t in range(1, T + 1))
        np.testing.assert_allclose(o.get(o.X), x0 - lr * g[0] * coef, rtol=1e-12)


@pytest.mark.parametrize("comp", [SIGN, TOPK])
@pytest.mark.parametrize("dtype,tol", [(np.float64, 1e-12), (np.float32, 2e-6)])
def test_size_one_tensors_reduce_to_momentum_sgd(comp, dtype, tol):
    """For a tensor of one element ||v||_1/1 sign(v) = v and top-1-of-1 = v: the real compressors are
    the identity, so the whole method must reproduce plain momentum SGD."""
    K, d = 2, 24
    sizes = [1] * d
    x0, gs = rand_sizes_grads(K, sizes, 6, dtype, scale=1.0)
    o = Oracle(K, sizes, x0, compressor=comp, momentum=0.9, avg_period=3, dtype=dtype)
    for g in gs:
        o.step(g, 0.1)
    x_ref, m_ref = momentum_sgd_numpy(x0, gs, K, 0.9, 0.1)
    np.testing.assert_allclose(o.get(o.X), x_ref, rtol=tol, atol=tol)
    np.testing.assert_allclose(o.get_all(o.M), m_ref, rtol=tol, atol=tol)
    assert np.all(o.get_all(o.E) == 0) and np.all(o.get(o.E_SRV) == 0)


def aux(o):
    """x~ = x - (e + mean_k e^(k))  (Section 2, Gradient Mismatch)."""
    return o.get(o.X).astype(np.float64) - (o.get(o.E_SRV).astype(np.float64)
                                             + o.get_all(o.E).astype(np.float64).mean(axis=0))


@pytest.mark.parametrize("comp", [SIGN, TOPK, IDENTITY])
@pytest.mark.parametrize("mode", [EF, SAEF])
@pytest.mark.parametrize("p", [0, 1, 3])
@pytest.mark.parametrize("dc", [0, 1])
def test_auxiliary_variable_identity_and_telescoping(comp, mode, p, dc):
    """Eq. 3 / Appendix A: x~_{t+1} = x~_t - (eta_t/K) sum_k m_{t+1}^(k) for any compressor, with or
    without error averaging; summed over t: x_0 - x_T = sum_t C(Delta_{t+1}) and
    sum_t C(Delta_{t+1}) + e_T + mean_k e_T^(k) = sum_t eta_t mean_k m_{t+1}^(k)."""
    K, sizes, steps = 3, [1, 7, 32, 65, 200], 9
    x0, gs = rand_sizes_grads(K, sizes, steps, np.float64)
    o = Oracle(K, sizes, x0, compressor=comp, server_compress=dc, mode=mode, avg_period=p, momentum=0.9,
               weight_decay=1e-3, topk_num=1, topk_den=10, dtype=np.float64)
    lrs = [0.1, 0.1, 0.05, 0.2, 0.1, 0.01, 0.1, 0.3, 0.1]
    applied = np.zeros_like(x0)
    mom_sum = np.zeros_like(x0)
    xt = aux(o)
    np.testing.assert_array_equal(xt, x0)
    for g, lr in zip(gs, lrs):
        x_before = o.get(o.X)
        o.step(g, lr)
        m = o.get_all(o.M)
        xt_new = aux(o)
        np.testing.assert_allclose(xt_new, xt - lr * m.mean(axis=0), rtol=0, atol=1e-13)
        xt = xt_new
        cs = o.get(o.C_DELTA_SRV)
        np.testing.assert_array_equal(o.get(o.X), x_before - cs)          # re-update
        applied += cs
        mom_sum += lr * m.mean(axis=0)
    np.testing.assert_allclose(x0 - o.get(o.X), applied, atol=1e-13)
    np.testing.assert_allclose(applied + o.get(o.E_SRV) + o.get_all(o.E).mean(axis=0), mom_sum, atol=1e-13)
    if not dc:
        assert np.all(o.get(o.E_SRV) == 0)


@pytest.mark.parametrize("comp", [SIGN, TOPK])
def test_telescoping_mu0_lr1_is_sum_of_gradients(comp):
    """mu = 0, eta = 1: applied updates + final errors = sum of worker-mean gradients."""
    K, sizes, steps = 4, [3, 50, 129], 8
    x0, gs = rand_sizes_grads(K, sizes, steps, np.float64)
    o = Oracle(K, sizes, x0, compressor=comp, avg_period=0, momentum=0.0, topk_num=1, topk_den=8, dtype=np.float64)
    for g in gs:
        o.step(g, 1.0)
    lhs = (x0 - o.get(o.X)) + o.get(o.E_SRV) + o.get_all(o.E).mean(axis=0)
    np.testing.assert_allclose(lhs, sum(g.mean(axis=0) for g in gs), atol=1e-13)


def np_scaled_sign(v):
    return np.abs(v).mean() * np.where(v >= 0, 1.0, -1.0)


def np_topk(v, kk):
    thr = np.sort(np.abs(v))[::-1][kk - 1]
    return np.where((np.abs(v) >= thr) & (v != 0), v, 0.0)


@pytest.mark.parametrize("comp", [SIGN, TOPK])
def test_first_iteration_is_plain_compressed_sgd(comp):
    """Zero error, EF mode (no step-ahead), first iteration: x_1 = x_0 - C(mean_k C(eta g^(k)))."""
    K, sizes = 3, [10, 64, 5]
    x0, gs = rand_sizes_grads(K, sizes, 1, np.float64)
    o = Oracle(K, sizes, x0, compressor=comp, mode=EF, momentum=0.9, topk_num=1, topk_den=5, dtype=np.float64)
    o.step(gs[0], 0.1)
    off = np.concatenate([[0], np.cumsum(sizes)])
    x1 = x0.copy()
    for j, n in enumerate(sizes):
        sl = slice(off[j], off[j + 1])
        f = np_scaled_sign if comp == SIGN else (lambda v: np_topk(v, max(1, len(v) // 5)))
        cw = np.stack([f(0.1 * gs[0][k, sl]) for k in range(K)])
        x1[sl] = x0[sl] - f(cw.sum(axis=0) / K)
    np.testing.assert_allclose(o.get(o.X), x1, rtol=1e-12, atol=1e-15)


def test_one_full_step_against_numpy_restatement():
    """Second iteration (non-zero errors) of the SAEF branch with weight decay, written independently
    in numpy from Algorithm 1: pins the step-ahead point, the coupled weight decay, Delta = e + eta m,
    the worker and server error updates and the worker-axis mean."""
    K, sizes = 4, [6, 40, 33]
    mu, lam = 0.8, 1e-2
    x0, gs = rand_sizes_grads(K, sizes, 3, np.float64, scale=1.0)
    off = np.concatenate([[0], np.cumsum(sizes)])
    for mode in (EF, SAEF):
        o = Oracle(K, sizes, x0, compressor=SIGN, mode=mode, momentum=mu, weight_decay=lam, dtype=np.float64)
        x, m, e, es = x0.copy(), np.zeros((K, x0.size)), np.zeros((K, x0.size)), np.zeros(x0.size)
        for g, lr in zip(gs, (0.1, 0.2, 0.05)):
            o.step(g, lr)
            xh = x[None, :] - e if mode == SAEF else np.broadcast_to(x, e.shape)
            m = mu * m + (g + lam * xh)
            D = e + lr * m
            c = np.zeros_like(D)
            for j in range(len(sizes)):
                sl = slice(off[j], off[j + 1])
                for k in range(K):
                    c[k, sl] = np_scaled_sign(D[k, sl])
            e = D - c
            Ds = es + c.mean(axis=0)
            cs = np.concatenate([np_scaled_sign(Ds[off[j]:off[j + 1]]) for j in range(len(sizes))])
            es = Ds - cs
            x = x - cs
            np.testing.assert_allclose(o.get_all(o.M), m, rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(o.get_all(o.DELTA), D, rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(o.get_all(o.E), e, rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(o.get(o.E_SRV), es, rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(o.get(o.X), x, rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(o.step_ahead(2), x - e[2] if mode == SAEF else x, rtol=1e-11, atol=1e-13)


def test_saef_equals_ef_without_weight_decay():
    """The two branches differ only in where the gradient is evaluated; with externally supplied
    gradients and lambda = 0 they coincide."""
    K, sizes = 2, [9, 70]
    x0, gs = rand_sizes_grads(K, sizes, 5, np.float32)
    a = Oracle(K, sizes, x0, mode=EF)
    b = Oracle(K, sizes, x0, mode=SAEF)
    for g in gs:
        a.step(g, 0.1)
        b.step(g, 0.1)
    np.testing.assert_array_equal(a.get(a.X), b.get(b.X))
    np.testing.assert_array_equal(a.get_all(a.E), b.get_all(b.E))


@pytest.mark.parametrize("comp", [SIGN, TOPK])
def test_error_averaging_schedule_and_invariants(comp):
    """Averaging happens in the pre-step of iteration t when (t+1) mod p = 0; it leaves mean_k e^(k)
    unchanged and zeroes the spread; p = 0 (infinity) never averages."""
    K, sizes, p = 4, [20, 100], 3
    x0, gs = rand_sizes_grads(K, sizes, 9, np.float64)
    o = Oracle(K, sizes, x0, compressor=comp, avg_period=p, dtype=np.float64)
    never = Oracle(K, sizes, x0, compressor=comp, avg_period=0, dtype=np.float64)
    for g in gs:
        o.step(g, 0.1)
        never.step(g, 0.1)
        e = o.get_all(o.E)
        raw = o.get_all(o.DELTA) - o.get_all(o.C_DELTA)        # e_{t+1}^(k) before the pre-step
        np.testing.assert_allclose(e.mean(axis=0), raw.mean(axis=0), atol=1e-15)
        spread = ((e - e.mean(axis=0)) ** 2).sum()
        if (o.iteration + 1) % p == 0:
            assert spread == 0.0
        else:
            assert spread > 0.0
            np.testing.assert_array_equal(e, raw)
        en = never.get_all(never.E)
        assert ((en - en.mean(axis=0)) ** 2).sum() > 0.0


@pytest.mark.parametrize("comp", [SIGN, TOPK])
@pytest.mark.parametrize("K", [2, 4])
def test_identical_workers_equal_single_worker(comp, K):
    """K workers fed the same gradient behave as one (K a power of two keeps the mean exact in fp32)."""
    sizes = [13, 64, 100]
    x0, gs = rand_sizes_grads(1, sizes, 6, np.float32)
    one = Oracle(1, sizes, x0, compressor=comp, avg_period=2, topk_num=1, topk_den=10)
    many = Oracle(K, sizes, x0, compressor=comp, avg_period=2, topk_num=1, topk_den=10)
    for g in gs:
        one.step(g, 0.1)
        many.step(np.repeat(g, K, axis=0), 0.1)
    np.testing.assert_array_equal(one.get(one.X), many.get(many.X))
    np.testing.assert_array_equal(one.get(one.E_SRV), many.get(many.E_SRV))
    for k in range(K):
        np.testing.assert_array_equal(one.get(one.E, 0), many.get(many.E, k))


def test_single_worker_server_sign_is_noop_at_first_step():
    """K = 1, e = 0: the server sees C(Delta^(1)) whose entries all have magnitude s, so C(C(v)) = C(v)."""
    sizes = [50, 7]
    x0, gs = rand_sizes_grads(1, sizes, 1, np.float64)
    o = Oracle(1, sizes, x0, compressor=SIGN, dtype=np.float64)
    o.step(gs[0], 0.1)
    np.testing.assert_allclose(o.get(o.C_DELTA_SRV), o.get(o.C_DELTA, 0), rtol=1e-12)
    np.testing.assert_allclose(o.get(o.E_SRV), 0, atol=1e-15)


def test_float_run_tracks_double_run():
    """The pinned fp32 instantiation follows the fp64 one (identity compressor: no discrete decisions)."""
    K, sizes = 3, [11, 90]
    x0, gs = rand_sizes_grads(K, sizes, 10, np.float32)
    a = Oracle(K, sizes, x0, compressor=IDENTITY, weight_decay=1e-3)
    b = Oracle(K, sizes, x0.astype(np.float64), compressor=IDENTITY, weight_decay=1e-3, dtype=np.float64)
    for g in gs:
        a.step(g, 0.1)
        b.step(g.astype(np.float64), 0.1)
    np.testing.assert_allclose(a.get(a.X), b.get(b.X), rtol=1e-5, atol=1e-6)


def test_float_sign_step_matches_double_where_signs_agree():
    """One fp32 sign step against the fp64 run: scales within float rounding, signs identical away from 0."""
    K, sizes = 2, [300, 31]
    x0, gs = rand_sizes_grads(K, sizes, 1, np.float32)
    a = Oracle(K, sizes, x0)
    b = Oracle(K, sizes, x0.astype(np.float64), dtype=np.float64)
    a.step(gs[0], 0.1)
    b.step(gs[0].astype(np.float64), 0.1)
    np.testing.assert_allclose(a.get_all(a.SCALES), b.get_all(b.SCALES), rtol=1e-6)
    np.testing.assert_allclose(a.get(a.SCALES_SRV), b.get(b.SCALES_SRV), rtol=1e-6)
    np.testing.assert_allclose(a.get(a.X), b.get(b.X), rtol=1e-5, atol=1e-7)


def test_thread_count_does_not_change_bits():
    K, sizes = 4, [100, 3, 64, 1000]
    x0, gs = rand_sizes_grads(K, sizes, 4, np.float32)
    for comp in (SIGN, TOPK):
        runs = []
        for th in (1, 3):
            o = Oracle(K, sizes, x0, compressor=comp, avg_period=2, threads=th, weight_decay=1e-4)
            for g in gs:
                o.step(g, 0.1)
            runs.append((o.get(o.X), o.get_all(o.E), o.get_all(o.M)))
        for u, v in zip(*runs):
            np.testing.assert_array_equal(u, v)


def test_range_flag_and_bad_config():
    sizes = [4]
    x0 = np.zeros(4, dtype=np.float32)
    o = Oracle(1, sizes, x0)
    o.step(np.array([[1.0, np.inf, 0.0, 0.0]], dtype=np.float32), 0.1)
    assert o.range_flag
    with pytest.raises(ValueError):
        Oracle(0, sizes, x0)
    with pytest.raises(ValueError):
        Oracle(1, [0], np.zeros(0, dtype=np.float32))


# ------------------------------------------------------------------------------------------------
# randomised property checks (hypothesis): the identities must hold for any shape and schedule
# ------------------------------------------------------------------------------------------------
from hypothesis import given, settings, strategies as st


@settings(max_examples=40, deadline=None)
@given(K=st.integers(1, 6), sizes=st.lists(st.integers(1, 300), min_size=1, max_size=5), comp=st.sampled_from([SIGN, TOPK]),
       mode=st.sampled_from([EF, SAEF]), p=st.integers(0, 4), dc=st.integers(0, 1), steps=st.integers(1, 6),
       seed=st.integers(0, 10 ** 6), mu=st.sampled_from([0.0, 0.5, 0.9]), lam=st.sampled_from([0.0, 1e-3]))
def test_auxiliary_identity_random_configurations(K, sizes, comp, mode, p, dc, steps, seed, mu, lam):
    """Eq. 3 per step and the telescoped sum x_0 - x_T = sum_t C(Delta_t), fp64, random configurations."""
    x0, gs = rand_sizes_grads(K, sizes, steps, np.float64, seed=seed)
    o = Oracle(K, sizes, x0, compressor=comp, server_compress=dc, mode=mode, avg_period=p, momentum=mu, weight_decay=lam,
               topk_num=1, topk_den=7, dtype=np.float64)
    xt = aux(o)
    applied = np.zeros_like(x0)
    for g in gs:
        o.step(g, 0.1)
        m = o.get_all(o.M)
        xt_new = aux(o)
        np.testing.assert_allclose(xt_new, xt - 0.1 * m.mean(axis=0), rtol=0, atol=1e-12)
        xt = xt_new
        applied += o.get(o.C_DELTA_SRV)
        # Assumption 4 for every worker tensor: ||C(v) - v||^2 <= ||v||^2
        D, c = o.get_all(o.DELTA), o.get_all(o.C_DELTA)
        assert ((D - c) ** 2).sum() <= (D ** 2).sum() * (1 + 1e-12) + 1e-300
    np.testing.assert_allclose(x0 - o.get(o.X), applied, atol=1e-12)


@settings(max_examples=30, deadline=None)
@given(n=st.integers(1, 400), scale_exp=st.integers(-30, 20), seed=st.integers(0, 10 ** 6))
def test_fixed_point_l1_random(n, scale_exp, seed):
    """Exact L1 against rational arithmetic for random magnitudes (including values >= 1 and tiny ones)."""
    rng = np.random.default_rng(seed)
    v = (rng.standard_normal(n) * 2.0 ** scale_exp).astype(np.float32)
    S, rg = so.l1_fixed(v)
    if np.all(np.abs(v) < 2.0 ** 32):
        assert not rg and S == _exact_fixed_sum(v)
    else:
        assert rg


# ------------------------------------------------------------------------------------------------
# local steps (Section 2: the model difference communicated every H iterations)
# ------------------------------------------------------------------------------------------------
def quad_problem(d, seed):
    """f_k(y) = 0.5 y'A_k y - b_k'y with A_k symmetric positive definite: gradient A_k y - b_k."""
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((d, d)) * 0.1
    return Q @ Q.T + 0.5 * np.eye(d), rng.standard_normal(d)


@pytest.mark.parametrize("comp", [SIGN, TOPK, IDENTITY])
def test_local_steps_period_one_is_algorithm_1(comp):
    """H = 1 communicates every iteration: bit for bit the run without local steps."""
    K, sizes = 3, [9, 64, 130]
    x0, gs = rand_sizes_grads(K, sizes, 5, np.float32)
    a = Oracle(K, sizes, x0, compressor=comp, momentum=0.9, weight_decay=1e-3, topk_den=10)
    b = Oracle(K, sizes, x0, compressor=comp, momentum=0.9, weight_decay=1e-3, topk_den=10, local_steps=1)
    for g in gs:
        a.step(g, 0.1); b.step(g, 0.1)
    for w in (a.X, a.E_SRV):
        np.testing.assert_array_equal(a.get(w), b.get(w))
    np.testing.assert_array_equal(a.get_all(a.E), b.get_all(b.E))


@pytest.mark.parametrize("H", [2, 3, 5])
def test_local_steps_single_worker_identity_is_momentum_sgd(H):
    """K = 1, C = identity: the gradient point y = x - e^(1) follows plain momentum SGD with weight decay
    (m <- mu m + grad f(y) + lambda y, y <- y - eta m) whatever the period; x itself moves only when communicating."""
    d, steps, mu, lr, lam = 12, 11, 0.9, 0.07, 1e-2
    A, b = quad_problem(d, 3)
    x0 = np.random.default_rng(5).standard_normal(d)
    o = Oracle(1, [5, 7], x0, compressor=IDENTITY, momentum=mu, weight_decay=lam, dtype=np.float64, local_steps=H)
    y, m = x0.copy(), np.zeros(d)
    for t in range(steps):
        pt = o.step_ahead(0)
        np.testing.assert_allclose(pt, y, rtol=0, atol=1e-12)
        x_before = o.get(o.X)
        o.step((A @ pt - b)[None, :], lr)
        m = mu * m + (A @ y - b + lam * y)           # coupled L2 at the point where the gradient is taken
        y = y - lr * m
        if (t + 1) % H:
            np.testing.assert_array_equal(o.get(o.X), x_before)          # nothing was communicated
        else:
            np.testing.assert_allclose(o.get(o.X), y, rtol=0, atol=1e-12)   # identity: no error is left
            assert np.all(o.get(o.E, 0) == 0)


@pytest.mark.parametrize("H", [2, 4])
def test_local_steps_identity_is_periodic_model_averaging(H):
    """C = identity, K workers with different objectives: every worker runs H momentum steps on its own
    copy of the model, then the copies are averaged (local SGD with periodic averaging, written out
    independently in numpy)."""
    K, d, rounds, mu, lr = 3, 10, 3, 0.8, 0.05
    probs = [quad_problem(d, 10 + k) for k in range(K)]
    x0 = np.random.default_rng(6).standard_normal(d)
    o = Oracle(K, [4, 6], x0, compressor=IDENTITY, momentum=mu, dtype=np.float64, local_steps=H)
    xs = [x0.copy() for _ in range(K)]
    ms = [np.zeros(d) for _ in range(K)]
    for r in range(rounds):
        for h in range(H):
            g = np.stack([probs[k][0] @ o.step_ahead(k) - probs[k][1] for k in range(K)])
            o.step(g, lr)
            for k in range(K):
                ms[k] = mu * ms[k] + (probs[k][0] @ xs[k] - probs[k][1])
                xs[k] = xs[k] - lr * ms[k]
        avg = np.mean(xs, axis=0)
        xs = [avg.copy() for _ in range(K)]
        np.testing.assert_allclose(o.get(o.X), avg, rtol=0, atol=1e-12)


@pytest.mark.parametrize("comp", [SIGN, TOPK])
@pytest.mark.parametrize("dc", [0, 1])
@pytest.mark.parametrize("H", [2, 3])
def test_local_steps_auxiliary_identity(comp, dc, H):
    """Eq. 3 holds at every iteration, communicating or not: x~ = x - (e + mean_k e^(k)) moves by
    -(eta/K) sum_k m^(k); a local iteration leaves x, the server error and the messages alone."""
    K, sizes, steps = 3, [1, 7, 32, 65, 200], 10
    x0, gs = rand_sizes_grads(K, sizes, steps, np.float64)
    o = Oracle(K, sizes, x0, compressor=comp, server_compress=dc, momentum=0.9, weight_decay=1e-3, topk_den=10,
               dtype=np.float64, local_steps=H)
    xt = aux(o)
    for t, g in enumerate(gs):
        lr = 0.1 if t % 2 else 0.05
        x_before, es_before, e_before = o.get(o.X), o.get(o.E_SRV), o.get_all(o.E)
        o.step(g, lr)
        m = o.get_all(o.M)
        xt_new = aux(o)
        np.testing.assert_allclose(xt_new, xt - lr * m.mean(axis=0), rtol=0, atol=1e-13)
        xt = xt_new
        if (t + 1) % H:
            np.testing.assert_array_equal(o.get(o.X), x_before)
            np.testing.assert_array_equal(o.get(o.E_SRV), es_before)
            np.testing.assert_allclose(o.get_all(o.E), e_before + lr * m, rtol=0, atol=1e-15)
        else:
            np.testing.assert_array_equal(o.get(o.X), x_before - o.get(o.C_DELTA_SRV))


def test_local_steps_rejects_ef_and_averaging():
    x0 = np.zeros(12, np.float32)
    with pytest.raises(ValueError):
        Oracle(2, [5, 7], x0, mode=EF, local_steps=2)
    with pytest.raises(ValueError):
        Oracle(2, [5, 7], x0, avg_period=4, local_steps=2)
