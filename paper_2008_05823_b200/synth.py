"""Seeded synthetic inputs (gradients, initial parameters) that stand in for back-propagation on the
paper's CIFAR-100 / ImageNet runs.  Holds none of the method's arithmetic.

Every value is a pure function of (seed, iteration t, worker k, flat element index i) through a
counter-based 64-bit integer hash, so that the numpy generator here and the CUDA generator
(csrc/synth_gen.cu, `fill_grads_device`) produce identical bits:

    key(seed, t, k)  = mix64(mix64(seed + C0) + t*C1 + k*C2)
    h_r(i)           = mix64(key + (4 i + r) * GAMMA),        r = 0..3   (sixteen 16-bit lanes)
    z                = (sum of lanes 0..11  -  393210) / 65536            Irwin-Hall, unit variance, exact in fp32
    g                = fp32(s_j) * z   [ * outlier_mult  if lane 12 < outlier_per_65536 ]

mix64 is the splitmix64 finaliser.  s_j = 10^(lo + (hi-lo) u_j) is computed here in double and rounded
to fp32 once; both generators read it from a table.
"""
import ctypes as C
import os

import numpy as np

MASK = (1 << 64) - 1
C0 = 0x5AE05823C0FFEE01
C1 = 0xD1342543DE82EF95
C2 = 0xA0761D6478BD642F
GAMMA = 0x9E3779B97F4A7C15
M1 = 0xBF58476D1CE4E5B9
M2 = 0x94D049BB133111EB
T_X0 = (1 << 40) + 1          # "iteration" ids of the non-gradient streams
T_SCALE = (1 << 40) + 2


def mix64_int(z: int) -> int:
    z &= MASK
    z = ((z ^ (z >> 30)) * M1) & MASK
    z = ((z ^ (z >> 27)) * M2) & MASK
    return z ^ (z >> 31)


def stream_key(seed: int, t: int, k: int) -> int:
    return mix64_int(mix64_int(seed + C0) + t * C1 + k * C2)


def _mix64_np(z):
    z = (z ^ (z >> np.uint64(30))) * np.uint64(M1)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(M2)
    return z ^ (z >> np.uint64(31))


def _unit_normal_and_lane12(key: int, i0: int, count: int):
    """z (float32, exact) and the 16-bit outlier lane for flat indices i0 .. i0+count-1."""
    with np.errstate(over="ignore"):
        i = np.arange(i0, i0 + count, dtype=np.uint64)
        total = np.zeros(count, dtype=np.int64)
        lane12 = None
        for r in range(4):
            h = _mix64_np(np.uint64(key) + (i * np.uint64(4) + np.uint64(r)) * np.uint64(GAMMA))
            if r < 3:
                for s in (0, 16, 32, 48):
                    total += ((h >> np.uint64(s)) & np.uint64(0xFFFF)).astype(np.int64)
            else:
                lane12 = (h & np.uint64(0xFFFF)).astype(np.int64)
    z = (total - 393210).astype(np.float32) * np.float32(1.0 / 65536.0)
    return z, lane12


def tensor_scales(seed: int, num_tensors: int, lo: float, hi: float) -> np.ndarray:
    """Per-tensor gradient scale s_j, log-uniform in [10^lo, 10^hi], float32."""
    out = np.empty(num_tensors, dtype=np.float32)
    for j in range(num_tensors):
        u = (stream_key(seed, T_SCALE, j) >> 11) / float(1 << 53)
        out[j] = np.float32(10.0 ** (lo + (hi - lo) * u))
    return out


def _elem_scales(tensor_sizes, scales, i0, count):
    sizes = np.asarray(tensor_sizes, dtype=np.int64)
    ends = np.cumsum(sizes)
    j = np.searchsorted(ends, np.arange(i0, i0 + count, dtype=np.int64), side="right")
    return scales[j]


def grads_numpy(seed, t, num_workers, tensor_sizes, scales, outlier_per_65536=0, outlier_mult=1.0,
                chunk=1 << 22) -> np.ndarray:
    """[K][d] float32 gradients of iteration t."""
    d = int(np.sum(np.asarray(tensor_sizes, dtype=np.int64)))
    out = np.empty((num_workers, d), dtype=np.float32)
    scales = np.asarray(scales, dtype=np.float32)
    om = np.float32(outlier_mult)
    for k in range(num_workers):
        key = stream_key(seed, t, k)
        for i0 in range(0, d, chunk):
            cnt = min(chunk, d - i0)
            z, lane12 = _unit_normal_and_lane12(key, i0, cnt)
            g = _elem_scales(tensor_sizes, scales, i0, cnt) * z
            if outlier_per_65536 > 0:
                g = np.where(lane12 < outlier_per_65536, g * om, g).astype(np.float32)
            out[k, i0:i0 + cnt] = g
    return out


def x0_numpy(seed, d, chunk=1 << 22) -> np.ndarray:
    """Initial parameters x_0 = 0.05 z from their own stream."""
    out = np.empty(d, dtype=np.float32)
    key = stream_key(seed, T_X0, 0)
    for i0 in range(0, d, chunk):
        cnt = min(chunk, d - i0)
        z, _ = _unit_normal_and_lane12(key, i0, cnt)
        out[i0:i0 + cnt] = np.float32(0.05) * z
    return out


def workload_scales(w, seed):
    return tensor_scales(seed, w.num_tensors, w.log10_scale_lo, w.log10_scale_hi)


def workload_grads_numpy(w, seed, t, scales=None, num_workers=None, tensor_sizes=None):
    if scales is None:
        scales = workload_scales(w, seed)
    return grads_numpy(seed, t, num_workers or w.num_workers, tensor_sizes or w.tensor_sizes, scales,
                       w.outlier_per_65536, w.outlier_mult)


# ---------------------------------------------------------------------------------------------------
# CUDA generator (same bits), for workloads too large to generate on the host.
_glib = None


def _gen_lib():
    global _glib
    if _glib is None:
        path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsae_synth.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2008_05823_b200.build` first")
        L = C.CDLL(path)
        L.sae_synth_fill.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_uint64, C.c_uint64, C.c_uint32, C.c_float, C.c_float, C.c_void_p]
        L.sae_synth_fill.restype = C.c_int
        _glib = L
    return _glib


class DeviceGenerator:
    """Fills device buffers with the same values as `grads_numpy` / `x0_numpy`."""

    def __init__(self, tensor_sizes, scales, device="cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        sizes = np.asarray(tensor_sizes, dtype=np.int64)
        self.d = int(sizes.sum())
        self.T = len(sizes)
        self.ends = torch.from_numpy(np.cumsum(sizes)).to(self.device)
        self.scales = torch.from_numpy(np.asarray(scales, dtype=np.float32)).to(self.device)
        self.ones = torch.ones(self.T, dtype=torch.float32, device=self.device)

    def _fill(self, out, rows, seed, t, scales, outlier_per_65536, outlier_mult, post_mult):
        torch = self.torch
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() == rows * self.d
        stream = torch.cuda.current_stream(self.device).cuda_stream
        rc = _gen_lib().sae_synth_fill(out.data_ptr(), self.d, rows, self.T, self.ends.data_ptr(), scales.data_ptr(),
                                       mix64_int(seed + C0), t, outlier_per_65536, outlier_mult, post_mult,
                                       C.c_void_p(stream))
        if rc != 0:
            raise RuntimeError(f"sae_synth_fill failed with CUDA error {rc}")
        return out

    def grads(self, out, num_workers, seed, t, outlier_per_65536=0, outlier_mult=1.0):
        return self._fill(out, num_workers, seed, t, self.scales, outlier_per_65536, outlier_mult, 1.0)

    def x0(self, out, seed):
        return self._fill(out, 1, seed, T_X0, self.ones, 0, 1.0, 0.05)


def grads_numpy_range(seed, t, k, i0, count, scale, outlier_per_65536=0, outlier_mult=1.0):
    """Gradient entries i0 .. i0+count-1 (flat caller-layout indices, all inside one tensor of scale
    `scale`) of worker k at iteration t: lets a test reproduce single tensors of a large workload."""
    z, lane12 = _unit_normal_and_lane12(stream_key(seed, t, k), i0, count)
    g = np.float32(scale) * z
    if outlier_per_65536 > 0:
        g = np.where(lane12 < outlier_per_65536, g * np.float32(outlier_mult), g).astype(np.float32)
    return g


def x0_numpy_range(seed, i0, count):
    z, _ = _unit_normal_and_lane12(stream_key(seed, T_X0, 0), i0, count)
    return np.float32(0.05) * z
