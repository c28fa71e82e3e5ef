"""The allocation-free entry point `sae_sign_compress_noalloc` (for callers that may not call cudaMalloc:
code living inside another framework's memory pool, plug-ins that only get their input and output
buffers, loops that cannot afford a device-wide synchronising allocation) against two references: the CPU
oracle's Eq. 2 (scale and sign words, bit for bit -- the tolerance of every other parity test here) and the
handle-based path.  With one worker, mu = 0, lr = 1 and zero initial state the first `sae_step` compresses
exactly the gradient it is given, so its scales and sign words are C(v) of Eq. 2 as well.
Runs last so that a failure here cannot hide the other tests."""
import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
import scale_cases

pytestmark = pytest.mark.gpu


def reference_through_handle(v):
    import torch
    n = v.numel()
    h = sb.Sae(1, [n], torch.zeros(n, device=v.device), compressor=sb.SIGN, momentum=0.0, avg_period=0)
    h.step(v.view(1, n), 1.0)
    h.sync()
    scale = h.get_state(sb.STATE_WORKER_SCALES, 0).cpu().numpy().copy()
    words = h.get_state(sb.STATE_WORKER_WORDS, 0).cpu().numpy().view(np.uint32).copy()
    h.close()
    return scale, words


def reference_through_oracle(v):
    """Eq. 2 on the host: the scale from the exact L1 sum, one bit per element (1 <-> v >= 0)."""
    vh = v.cpu().numpy()
    _, scale, _, rg = so.compress(so.SIGN, vh)
    return np.float32(scale), so.pack_signs(vh, [vh.size]), rg


def check_against_oracle(v, words, scale, flag, tag):
    import torch
    words.fill_(-1)
    sb.sign_compress_noalloc(v, words, scale, flag)
    torch.cuda.synchronize()
    exp_scale, exp_words, rg = reference_through_oracle(v)
    got_scale = scale.cpu().numpy()
    assert got_scale.view(np.uint32)[0] == np.array([exp_scale]).view(np.uint32)[0], (tag, got_scale, exp_scale)
    assert np.array_equal(words.cpu().numpy().view(np.uint32)[:exp_words.size], exp_words), tag
    if flag is not None:
        assert int(flag.item()) == int(rg), tag


def test_noalloc_matches_oracle_and_handle_path_on_two_calls_in_a_row():
    import torch
    gen = torch.Generator(device="cuda").manual_seed(5)
    for n in (1, 33, 4096, 5000, 3 * 4096, 1_000_003):
        # buffers are the caller's; allocate them before the calls under test
        words = torch.empty((n + 31) // 32, dtype=torch.int32, device="cuda")
        scale = torch.empty(1, dtype=torch.float32, device="cuda")
        flag = torch.empty(1, dtype=torch.int32, device="cuda")
        inputs = [torch.randn(n, device="cuda", generator=gen) * 1e-2,
                  torch.randn(n, device="cuda", generator=gen) * 30.0]
        inputs[1][::7] = 0.0
        for call, v in enumerate(inputs):           # two calls in a row share the scratch array
            words.fill_(-1)
            sb.sign_compress_noalloc(v, words, scale, flag)
            torch.cuda.synchronize()
            exp_scale, exp_words = reference_through_handle(v)
            got_scale = scale.cpu().numpy()
            assert got_scale.view(np.uint32)[0] == exp_scale.view(np.uint32)[0], (n, call, got_scale, exp_scale)
            assert np.array_equal(words.cpu().numpy().view(np.uint32), exp_words), (n, call)
            assert int(flag.item()) == 0
            o_scale, o_words, _ = reference_through_oracle(v)
            assert got_scale.view(np.uint32)[0] == np.array([o_scale]).view(np.uint32)[0], (n, call, got_scale, o_scale)
            assert np.array_equal(words.cpu().numpy().view(np.uint32), o_words), (n, call)


def test_noalloc_unaligned_input_and_no_range_flag():
    """Full tiles whose first element is 4-byte but not 16-byte aligned (a view one, two or three floats into
    an allocation: the lane-strided path instead of the 128-bit loads), and calls without a range flag."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(6)
    for n in (2 * 4096 + 5, 4 * 4096, 33):
        buf = torch.randn(n + 3, device="cuda", generator=gen) * 1e-2
        buf[::5] *= 300.0                                   # some magnitudes above 1
        words = torch.empty((n + 31) // 32, dtype=torch.int32, device="cuda")
        scale = torch.empty(1, dtype=torch.float32, device="cuda")
        flag = torch.empty(1, dtype=torch.int32, device="cuda")
        for shift in (1, 2, 3, 0):
            v = buf[shift:shift + n]
            assert v.data_ptr() % 16 == (4 * shift) % 16
            check_against_oracle(v, words, scale, flag, (n, shift))
            check_against_oracle(v, words, scale, None, (n, shift, "no flag"))


def test_noalloc_scale_truncates_the_exact_sum():
    """Tensors whose exact L1 sum gives different floats when truncated to 53 bits (the reading taken) and
    when rounded: the entry point follows the oracle and the exact rational arithmetic of the test."""
    import torch
    for n, top in ((8, 60), (8, 90), (4096, 62), (5000, 70), (3 * 4096 + 7, 93), (1 << 20, 66)):
        vh = scale_cases.discriminating_tensor(n, top, seed=n)
        S = scale_cases.fixed_sum(vh)
        v = torch.from_numpy(vh).cuda()
        words = torch.empty((n + 31) // 32, dtype=torch.int32, device="cuda")
        scale = torch.empty(1, dtype=torch.float32, device="cuda")
        flag = torch.empty(1, dtype=torch.int32, device="cuda")
        check_against_oracle(v, words, scale, flag, (n, top))
        got = scale.cpu().numpy()[0]
        assert got == scale_cases.scale_truncating(S, n) != scale_cases.scale_rounding(S, n), (n, top)


def test_noalloc_range_flag_and_size_limit():
    import torch
    n = 5000
    v = torch.ones(n, device="cuda")
    v[123] = float("inf")
    words = torch.empty((n + 31) // 32, dtype=torch.int32, device="cuda")
    scale = torch.empty(1, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    sb.sign_compress_noalloc(v, words, scale, flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1
    v[123] = 1.0
    sb.sign_compress_noalloc(v, words, scale, flag)      # the flag does not stick to the next call
    torch.cuda.synchronize()
    assert int(flag.item()) == 0 and float(scale.item()) == 1.0
    # beyond the fixed scratch capacity: rejected on the host, nothing launched
    limit = sb.noalloc_max_elements()
    assert limit == 8192 * 4096
    L = sb.lib()
    rc = L.sae_sign_compress_noalloc(v.data_ptr(), limit + 1, words.data_ptr(), scale.data_ptr(), None, None)
    assert rc == sb.ERR_TOO_LARGE
    assert b"scratch" in L.sae_strerror(rc)
    assert L.sae_sign_compress_noalloc(v.data_ptr(), 0, words.data_ptr(), scale.data_ptr(), None, None) == sb.ERR_INVALID_ARG
    assert L.sae_sign_compress_noalloc(None, 10, words.data_ptr(), scale.data_ptr(), None, None) == sb.ERR_INVALID_ARG
