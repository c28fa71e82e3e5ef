"""ctypes view of the CPU oracle (oracle/sae_oracle.cpp).

Test infrastructure: only the tests, the smoke check and the benchmark's CPU-baseline leg import this.
It performs no arithmetic of its own -- it marshals numpy arrays into the C functions.
"""
import ctypes as C
import os

import numpy as np

from . import build_oracle

IDENTITY, SIGN, TOPK = 0, 1, 2
EF, SAEF = 0, 1

_lib = None


def lib():
    global _lib
    if _lib is None:
        path = build_oracle.build()
        L = C.CDLL(path)
        for suf, ct in (("f32", C.c_float), ("f64", C.c_double)):
            getattr(L, f"sao_create_{suf}").restype = C.c_void_p
            getattr(L, f"sao_create_{suf}").argtypes = [
                C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double, C.c_double,
                C.c_uint32, C.c_uint32, C.c_int, C.c_void_p]
            getattr(L, f"sao_destroy_{suf}").argtypes = [C.c_void_p]
            getattr(L, f"sao_destroy_{suf}").restype = None
            getattr(L, f"sao_step_{suf}").argtypes = [C.c_void_p, C.c_void_p, C.c_double]
            getattr(L, f"sao_step_{suf}").restype = None
            getattr(L, f"sao_get_{suf}").argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p]
            getattr(L, f"sao_iteration_{suf}").argtypes = [C.c_void_p]
            getattr(L, f"sao_iteration_{suf}").restype = C.c_int64
            getattr(L, f"sao_range_flag_{suf}").argtypes = [C.c_void_p]
            getattr(L, f"sao_set_local_steps_{suf}").argtypes = [C.c_void_p, C.c_int]
            getattr(L, f"sao_get_tau_{suf}").argtypes = [C.c_void_p, C.c_int, C.c_void_p]
            getattr(L, f"sao_get_tau_{suf}").restype = None
            getattr(L, f"sao_compress_{suf}").argtypes = [
                C.c_int, C.c_void_p, C.c_int64, C.c_uint32, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.sao_l1_fixed_f32.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.sao_scale_from_fixed_f32.argtypes = [C.c_uint64, C.c_uint64, C.c_int64]
        L.sao_scale_from_fixed_f32.restype = C.c_float
        L.sao_topk_count.argtypes = [C.c_int64, C.c_uint32, C.c_uint32]
        L.sao_topk_count.restype = C.c_int64
        L.sao_pack_signs_f32.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.sao_pack_signs_f32.restype = C.c_int64
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


class Oracle:
    """One run of Algorithm 1.  dtype float32 = the pinned arithmetic, float64 = identity checks."""

    X, E_SRV, M, E, DELTA, C_DELTA, DELTA_SRV, C_DELTA_SRV, SCALES, SCALES_SRV = range(10)

    def __init__(self, num_workers, tensor_sizes, x0, compressor=SIGN, server_compress=1, mode=SAEF,
                 avg_period=0, momentum=0.9, weight_decay=0.0, topk_num=1, topk_den=100, threads=1,
                 dtype=np.float32, local_steps=1):
        self.dtype = np.dtype(dtype)
        self.suf = "f32" if self.dtype == np.float32 else "f64"
        self.K = int(num_workers)
        self.mode = mode
        self.sizes = np.ascontiguousarray(tensor_sizes, dtype=np.int64)
        self.T = len(self.sizes)
        self.d = int(self.sizes.sum())
        x0 = np.ascontiguousarray(x0, dtype=self.dtype)
        assert x0.shape == (self.d,)
        self.h = getattr(lib(), f"sao_create_{self.suf}")(
            self.K, self.T, _ptr(self.sizes), compressor, server_compress, mode, avg_period, float(momentum),
            float(weight_decay), topk_num, topk_den, threads, _ptr(x0))
        if not self.h:
            raise ValueError("oracle rejected the configuration")
        self.local_steps = int(local_steps)
        if getattr(lib(), f"sao_set_local_steps_{self.suf}")(self.h, self.local_steps) != 0:
            raise ValueError("local steps need the step-ahead branch without error averaging")

    def __del__(self):
        try:
            if getattr(self, "h", None):
                getattr(lib(), f"sao_destroy_{self.suf}")(self.h)
                self.h = None
        except Exception:      # interpreter shutdown
            pass

    def step(self, grads, lr):
        g = np.ascontiguousarray(grads, dtype=self.dtype)
        assert g.size == self.K * self.d
        getattr(lib(), f"sao_step_{self.suf}")(self.h, _ptr(g), float(lr))

    def get(self, which, worker=0):
        n = self.T if which in (self.SCALES, self.SCALES_SRV) else self.d
        out = np.empty(n, dtype=self.dtype)
        rc = getattr(lib(), f"sao_get_{self.suf}")(self.h, which, worker, _ptr(out))
        if rc != 0:
            raise ValueError("bad getter arguments")
        return out

    def get_all(self, which):
        return np.stack([self.get(which, k) for k in range(self.K)])

    def tau(self, worker):
        """Top-K threshold keys of the last step ([T] uint64); worker < 0 = server."""
        out = np.empty(self.T, dtype=np.uint64)
        getattr(lib(), f"sao_get_tau_{self.suf}")(self.h, worker, _ptr(out))
        return out

    @property
    def iteration(self):
        return int(getattr(lib(), f"sao_iteration_{self.suf}")(self.h))

    @property
    def range_flag(self):
        return bool(getattr(lib(), f"sao_range_flag_{self.suf}")(self.h))

    def step_ahead(self, worker):
        """The point where worker k evaluates its next gradient: x_t - e_t^(k) in the SAEF branch (one
        subtraction in the run's precision), x_t in the EF branch."""
        if self.mode == EF:
            return self.get(self.X)
        return self.get(self.X) - self.get(self.E, worker)


def compress(compressor, v, topk_num=1, topk_den=100):
    """C(v) on one tensor. Returns (c, scale, tau_key, range_flag)."""
    v = np.ascontiguousarray(v)
    suf = "f32" if v.dtype == np.float32 else "f64"
    c = np.empty_like(v)
    scale = np.zeros(1, dtype=v.dtype)
    tau = np.zeros(1, dtype=np.uint64)
    rg = getattr(lib(), f"sao_compress_{suf}")(compressor, _ptr(v), v.size, topk_num, topk_den, _ptr(c), _ptr(scale),
                                               _ptr(tau))
    return c, scale[0], int(tau[0]), bool(rg)


def l1_fixed(v):
    """sum_i floor(|v_i| 2^64) as a Python int, plus the range flag."""
    v = np.ascontiguousarray(v, dtype=np.float32)
    out = np.zeros(2, dtype=np.uint64)
    rg = lib().sao_l1_fixed_f32(_ptr(v), v.size, _ptr(out))
    return int(out[0]) | (int(out[1]) << 64), bool(rg)


def scale_from_fixed(S, n):
    return np.float32(lib().sao_scale_from_fixed_f32(S & ((1 << 64) - 1), S >> 64, n))


def topk_count(n, num, den):
    return int(lib().sao_topk_count(n, num, den))


def pack_signs(v, tensor_sizes):
    v = np.ascontiguousarray(v, dtype=np.float32)
    sizes = np.ascontiguousarray(tensor_sizes, dtype=np.int64)
    nw = int(((sizes + 31) // 32).sum())
    words = np.empty(nw, dtype=np.uint32)
    got = lib().sao_pack_signs_f32(_ptr(v), len(sizes), _ptr(sizes), _ptr(words))
    assert got == nw
    return words


def max_threads():
    return int(lib().sao_max_threads())
