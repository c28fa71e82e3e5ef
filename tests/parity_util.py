"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same bytes and
compare every piece of state element by element."""
import numpy as np

from oracle import sae_oracle as so
from paper_2008_05823_b200 import binding as sb

# Floating-point bar stated for this path: 1e-5 relative.  The two sides pin every rounding (fused ops,
# summation order, the exact L1), so the tests demand identical bits and only fall back to reporting
# the relative error when that fails.
RTOL = 1e-5


def assert_same(name, got, exp):
    got = np.asarray(got)
    exp = np.asarray(exp)
    assert got.shape == exp.shape, f"{name}: shape {got.shape} vs {exp.shape}"
    if got.dtype.kind == "f":
        same = (got.view(np.uint32) == exp.view(np.uint32)) | ((got == 0) & (exp == 0))
        if not same.all():
            bad = np.flatnonzero(~same.ravel())
            rel = np.abs(got.ravel()[bad] - exp.ravel()[bad]) / np.maximum(np.abs(exp.ravel()[bad]), 1e-30)
            raise AssertionError(f"{name}: {bad.size} of {got.size} floats differ (first at {bad[0]}: "
                                 f"{got.ravel()[bad[0]]!r} vs {exp.ravel()[bad[0]]!r}); max rel err {rel.max():.3e} "
                                 f"(stated bar {RTOL})")
    else:
        if not np.array_equal(got, exp):
            bad = np.flatnonzero(got.ravel() != exp.ravel())
            raise AssertionError(f"{name}: {bad.size} of {got.size} integers differ (first at {bad[0]}: "
                                 f"{got.ravel()[bad[0]]:#x} vs {exp.ravel()[bad[0]]:#x})")


def mask_words(selected, sizes):
    """Pack a boolean selection (caller layout) into the bit-word format."""
    out = []
    q = 0
    for n in sizes:
        bits = np.zeros(((n + 31) // 32) * 32, dtype=np.uint8)
        bits[:n] = selected[q:q + n]
        out.append(np.packbits(bits.reshape(-1, 32)[:, ::-1], axis=1).view(">u4").astype(np.uint32).ravel())
        q += n
    return np.concatenate(out)


def compare_state(gpu, orc, compressor, check_messages=True, tag=""):
    """gpu: binding.Sae, orc: oracle.Oracle (float32) after the same number of steps."""
    K, sizes = orc.K, orc.sizes
    cpu = lambda t: t.cpu().numpy()
    gpu.sync()
    assert gpu.iteration == orc.iteration
    assert_same(f"{tag} x", cpu(gpu.get_params()), orc.get(orc.X))
    assert_same(f"{tag} e_srv", cpu(gpu.get_state(sb.STATE_SERVER_ERROR)), orc.get(orc.E_SRV))
    for k in range(K):
        if gpu.keeps_momentum:      # with mu = 0 the library holds no momentum rows (m^(k) is the gradient term)
            assert_same(f"{tag} m[{k}]", cpu(gpu.get_state(sb.STATE_MOMENTUM, k)), orc.get(orc.M, k))
        assert_same(f"{tag} e[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_ERROR, k)), orc.get(orc.E, k))
        assert_same(f"{tag} step_ahead[{k}]", cpu(gpu.get_step_ahead(k)), orc.step_ahead(k))
    if not check_messages or orc.iteration == 0:
        return
    if compressor == so.SIGN:
        for k in range(K):
            assert_same(f"{tag} scales[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_SCALES, k)), orc.get(orc.SCALES, k))
            assert_same(f"{tag} words[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_WORDS, k)).view(np.uint32),
                        so.pack_signs(orc.get(orc.DELTA, k), sizes))
    elif compressor == so.TOPK:
        for k in range(K):
            assert_same(f"{tag} tau[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_TAU, k)).view(np.uint32).astype(np.uint64),
                        orc.tau(k))
            c = orc.get(orc.C_DELTA, k)
            sel = c != 0          # selected entries are never exact zeros
            assert_same(f"{tag} mask[{k}]", cpu(gpu.get_state(sb.STATE_WORKER_MASK, k)).view(np.uint32),
                        mask_words(sel, sizes))


def compare_server_messages(gpu, orc, compressor, server_compress, tag=""):
    cpu = lambda t: t.cpu().numpy()
    if not server_compress or orc.iteration == 0:
        return
    if compressor == so.SIGN:
        assert_same(f"{tag} scales_srv", cpu(gpu.get_state(sb.STATE_SERVER_SCALES)), orc.get(orc.SCALES_SRV))
        assert_same(f"{tag} words_srv", cpu(gpu.get_state(sb.STATE_SERVER_WORDS)).view(np.uint32),
                    so.pack_signs(orc.get(orc.DELTA_SRV), orc.sizes))
    elif compressor == so.TOPK:
        assert_same(f"{tag} tau_srv", cpu(gpu.get_state(sb.STATE_SERVER_TAU)).view(np.uint32).astype(np.uint64),
                    orc.tau(-1))
        cs = orc.get(orc.C_DELTA_SRV)
        assert_same(f"{tag} mask_srv", cpu(gpu.get_state(sb.STATE_SERVER_MASK)).view(np.uint32),
                    mask_words(cs != 0, orc.sizes))
