"""A failed initialisation cleans up after itself.  With SAE_DEBUG_FAIL_ALLOC=<n> (read by sae_init, testing
only) the n-th device allocation of that call reports an allocation failure without touching the allocator --
no GPU memory is exhausted to provoke it.  For every n up to the number of allocations the call makes, sae_init
must return SAE_ERR_NOMEM with no handle, give back everything it had allocated before (device memory, the
pinned status word, the second stream and its events), and leave the library usable."""
import os

import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from parity_util import compare_state

pytestmark = pytest.mark.gpu

CASES = [
    dict(K=4, sizes=[33, 4096, 5000], kw=dict(compressor=sb.SIGN, avg_period=1)),                 # small: rotating records
    dict(K=8, sizes=[33, 4096, 70_000], kw=dict(compressor=sb.TOPK, avg_period=1, topk_den=50)),  # second stream, two selects
    dict(K=8, sizes=[33, 4096, 70_000], kw=dict(compressor=sb.TOPK, avg_period=3, topk_den=50)),
    dict(K=2, sizes=[5000, (1 << 23) + 77], kw=dict(compressor=sb.SIGN, avg_period=0)),           # large: stored differences
    dict(K=4, sizes=[33, 4096, 5000], kw=dict(compressor=sb.TOPK, avg_period=2, shard=(1, 2))),   # a shard's tables
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"K{c['K']}-{c['kw']['compressor']}-p{c['kw']['avg_period']}")
def test_every_allocation_of_sae_init_may_fail(case):
    import torch
    K, sizes, kw = case["K"], case["sizes"], case["kw"]
    d = int(np.sum(sizes))
    x0 = torch.from_numpy(synth.x0_numpy(1, d)).cuda()
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    failed = 0
    for n in range(200):
        os.environ["SAE_DEBUG_FAIL_ALLOC"] = str(n)
        try:
            try:
                h = sb.Sae(K, sizes, x0, **kw)
            except sb.SaeError as err:
                assert err.status == sb.ERR_NOMEM, (n, err.status)
                failed += 1
                continue
        finally:
            del os.environ["SAE_DEBUG_FAIL_ALLOC"]
        h.close()                        # n is beyond the last allocation: the call went through
        break
    else:
        raise AssertionError("sae_init makes more than 200 allocations?")
    assert failed >= 20, failed          # tables, state, messages, records, scratch ...
    torch.cuda.synchronize()
    # everything was given back (the allocator may keep a little slack per freed block: allow 8 MB)
    assert torch.cuda.mem_get_info()[0] >= free0 - (8 << 20), (free0, torch.cuda.mem_get_info()[0])


def test_library_is_usable_after_failed_initialisations():
    import torch
    K, sizes = 4, [33, 4096, 5000]
    d = int(np.sum(sizes))
    x0 = synth.x0_numpy(1, d)
    os.environ["SAE_DEBUG_FAIL_ALLOC"] = "7"
    try:
        with pytest.raises(sb.SaeError):
            sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=1)
    finally:
        del os.environ["SAE_DEBUG_FAIL_ALLOC"]
    scales = synth.tensor_scales(1, len(sizes), -4.0, -1.0)
    orc = so.Oracle(K, sizes, x0, compressor=so.SIGN, avg_period=1)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=1)
    for t in range(3):
        g = synth.grads_numpy(1, t, K, sizes, scales)
        orc.step(g, 0.1)
        gpu.step(torch.from_numpy(g).cuda(), 0.1)
    compare_state(gpu, orc, so.SIGN, tag="after failed initialisations")
    gpu.close()
