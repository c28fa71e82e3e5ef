"""The allocation-free entry point `sae_sign_compress_noalloc` (for callers that may not call cudaMalloc:
code living inside another framework's memory pool, plug-ins that only get their input and output
buffers, loops that cannot afford a device-wide synchronising allocation) against the handle-based
path.  With one worker, mu = 0, lr = 1 and zero initial state the first `sae_step` compresses exactly
the gradient it is given, so its scales and sign words are C(v) of Eq. 2 for each tensor -- the values
the new entry point must reproduce bit for bit (the tolerance of every other parity test here).
Runs last so that a failure here cannot hide the other tests."""
import numpy as np
import pytest

from paper_2008_05823_b200 import binding as sb

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


def test_noalloc_matches_handle_path_on_two_calls_in_a_row():
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
