"""A bounded device wait that runs out.  The kernels' producers announce the bytes of every copy to an
mbarrier before they issue it; with SAE_DEBUG_DROP_COPY set, the copies of one chosen work item are announced
but never issued, so every warp waiting for that item polls until the handle's limit (SAE_WAIT_LIMIT_US, a few
milliseconds here) and gives up: the kernel returns by itself, the handle reports SAE_ERR_TIMEOUT at the next
sae_sync, nothing traps or faults, and the CUDA context stays usable -- a fresh handle on the same device then
matches the oracle bit for bit."""
import os
import time

import numpy as np
import pytest

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb
from paper_2008_05823_b200 import synth
from parity_util import compare_state

pytestmark = pytest.mark.gpu


def _run_until_timeout(K, sizes, p, drop, steps):
    import torch
    d = int(np.sum(sizes))
    x0 = torch.from_numpy(synth.x0_numpy(2, d)).cuda()
    scales = synth.tensor_scales(2, len(sizes), -4.0, -1.0)
    g = torch.from_numpy(synth.grads_numpy(2, 0, K, sizes, scales)).cuda()
    os.environ["SAE_DEBUG_DROP_COPY"] = str(drop)
    os.environ["SAE_WAIT_LIMIT_US"] = "3000"
    try:
        h = sb.Sae(K, sizes, x0, compressor=sb.SIGN, avg_period=p)
    finally:
        del os.environ["SAE_DEBUG_DROP_COPY"], os.environ["SAE_WAIT_LIMIT_US"]
    t0 = time.perf_counter()
    status = None
    for t in range(steps):
        h.step(g, 0.1)
        try:
            h.sync()
        except sb.SaeError as err:
            status = (t, err.status)
            break
    elapsed = time.perf_counter() - t0
    h.close()
    torch.cuda.synchronize()                      # the context is alive: no sticky CUDA error
    return status, elapsed


def _fresh_handle_is_exact(K, sizes, p):
    import torch
    d = int(np.sum(sizes))
    x0 = synth.x0_numpy(2, d)
    scales = synth.tensor_scales(2, len(sizes), -4.0, -1.0)
    orc = so.Oracle(K, sizes, x0, compressor=so.SIGN, avg_period=p, threads=4)
    gpu = sb.Sae(K, sizes, torch.from_numpy(x0).cuda(), compressor=sb.SIGN, avg_period=p)
    for t in range(3):
        g = synth.grads_numpy(2, t, K, sizes, scales)
        orc.step(g, 0.1)
        gpu.step(torch.from_numpy(g).cuda(), 0.1)
    compare_state(gpu, orc, so.SIGN, tag="after a timed-out handle")
    gpu.close()


def test_worker_pass_wait_runs_out():
    """Item 0 of the plain worker pass = (tile 0, worker 0), a full tile fetched by bulk copies (a problem above
    the small-problem limit: below it the worker pass makes no bulk copies)."""
    K, sizes, p = 4, [(1 << 22) + 3 * 4096, 5000], 0
    status, elapsed = _run_until_timeout(K, sizes, p, drop=0, steps=1)
    assert status == (0, sb.ERR_TIMEOUT), status
    assert elapsed < 10.0
    _fresh_handle_is_exact(K, sizes, p)


def test_folded_worker_pass_wait_runs_out():
    """One worker, p = 1: the second step runs the folded-averaging pass, whose element ranges are half tiles --
    the dropped index lies beyond the first step's items (one per tile) and beyond the server pass's tiles."""
    K, sizes, p = 1, [(1 << 24) + 4 * 4096, 5000, 2 * 4096], 1          # (above the small-problem limit)
    ntiles = (1 << 12) + 4 + 2 + 2
    status, elapsed = _run_until_timeout(K, sizes, p, drop=2 * ntiles - 2, steps=3)
    assert status == (1, sb.ERR_TIMEOUT), status
    assert elapsed < 10.0
    _fresh_handle_is_exact(K, sizes, p)


def test_server_pass_wait_runs_out():
    """Above the small-problem limit the server pass stages a full tile's server error through a bulk copy.
    Dropped index 2 = server tile 2 (full, first tile of the large tensor); for the worker pass index 2 is
    (tile 1, worker 0), a ragged tile that is not fetched by bulk copies, so only the server pass waits."""
    K, sizes, p = 2, [5000, (1 << 23) + 4096 * 3 + 77], 0
    status, elapsed = _run_until_timeout(K, sizes, p, drop=2, steps=1)
    assert status == (0, sb.ERR_TIMEOUT), status
    assert elapsed < 10.0
    _fresh_handle_is_exact(K, sizes, p)
