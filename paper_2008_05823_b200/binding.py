"""Thin ctypes binding of libsae.so (include/sae.h): argument marshalling only.  Every step of the path
runs in the library's CUDA kernels; torch is used here for device memory and streams.  There is no CPU
fallback: a missing library or a failing call raises.
"""
import ctypes as C
import os

import numpy as np

ABI_VERSION = 1
IDENTITY, SIGN, TOPK = 0, 1, 2
EF, SAEF = 0, 1
NUM_KERNELS = 12

(STATE_MOMENTUM, STATE_WORKER_ERROR, STATE_SERVER_ERROR, STATE_WORKER_SCALES, STATE_SERVER_SCALES,
 STATE_WORKER_WORDS, STATE_SERVER_WORDS, STATE_WORKER_TAU, STATE_SERVER_TAU, STATE_WORKER_MASK,
 STATE_SERVER_MASK, STATE_TOPK_FALLBACKS) = range(12)

OK, ERR_INVALID_ARG, ERR_NOMEM, ERR_CUDA, ERR_RANGE, ERR_TIMEOUT, ERR_ABI, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5, -6, -7

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsae.so")

EXPORTS = ["sae_init", "sae_step", "sae_step_host", "sae_get_params", "sae_get_params_host", "sae_get_step_ahead",
           "sae_get_state", "sae_iteration", "sae_num_params", "sae_num_words", "sae_sync", "sae_set_profiling",
           "sae_get_kernel_times", "sae_kernel_name", "sae_kernel_launches", "sae_destroy", "sae_strerror",
           "sae_last_cuda_error", "sae_sign_compress_noalloc", "sae_noalloc_max_elements", "sae_state_bytes",
           "sae_save_state", "sae_load_state", "sae_get_mismatch", "sae_init_shard", "sae_shard_export",
           "sae_shard_attach", "sae_shard_detach", "sae_step_begin", "sae_step_end", "sae_shard_set_avg_mode", "sae_avg_due",
           "sae_num_padded", "sae_avg_local_sum", "sae_avg_set", "sae_set_local_steps"]

SHARD_BLOB_BYTES = 1024


class SaeConfig(C.Structure):
    _fields_ = [("abi_version", C.c_uint32), ("num_workers", C.c_int32), ("num_tensors", C.c_int32),
                ("tensor_sizes", C.POINTER(C.c_int64)), ("compressor", C.c_int32), ("server_compress", C.c_int32),
                ("mode", C.c_int32), ("avg_period", C.c_int32), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("topk_num", C.c_uint32), ("topk_den", C.c_uint32), ("device", C.c_int32), ("stream", C.c_void_p)]


class SaeError(RuntimeError):
    def __init__(self, status, what, cuda_error=0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{what}: {lib().sae_strerror(status).decode()} ({status})"
        if cuda_error:
            msg += f", cudaError {cuda_error}"
        super().__init__(msg)


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2008_05823_b200.build` (needs nvcc); "
                               "there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
        L.sae_init.argtypes = [C.POINTER(SaeConfig), vp, C.POINTER(vp)]
        L.sae_step.argtypes = [vp, vp, f32]
        L.sae_step_host.argtypes = [vp, vp, f32]
        L.sae_get_params.argtypes = [vp, vp]
        L.sae_get_params_host.argtypes = [vp, vp]
        L.sae_get_step_ahead.argtypes = [vp, i32, vp]
        L.sae_get_state.argtypes = [vp, i32, i32, vp, C.c_size_t]
        for f in ("sae_iteration", "sae_num_params", "sae_num_words", "sae_kernel_launches"):
            getattr(L, f).argtypes = [vp]
            getattr(L, f).restype = i64
        L.sae_sync.argtypes = [vp]
        L.sae_set_profiling.argtypes = [vp, i32]
        L.sae_get_kernel_times.argtypes = [vp, vp, vp]
        L.sae_kernel_name.argtypes = [i32]
        L.sae_kernel_name.restype = C.c_char_p
        L.sae_destroy.argtypes = [vp]
        L.sae_destroy.restype = None
        L.sae_strerror.argtypes = [C.c_int]
        L.sae_strerror.restype = C.c_char_p
        L.sae_last_cuda_error.argtypes = [vp]
        L.sae_state_bytes.argtypes = [vp]
        L.sae_state_bytes.restype = i64
        L.sae_save_state.argtypes = [vp, vp, C.c_size_t]
        L.sae_load_state.argtypes = [vp, vp, C.c_size_t]
        L.sae_get_mismatch.argtypes = [vp, vp]
        L.sae_init_shard.argtypes = [C.POINTER(SaeConfig), i32, i32, vp, C.POINTER(vp)]
        L.sae_shard_export.argtypes = [vp, vp, C.c_size_t]
        L.sae_shard_attach.argtypes = [vp, vp, C.c_size_t]
        L.sae_shard_detach.argtypes = [vp]
        L.sae_step_begin.argtypes = [vp, vp, f32]
        L.sae_step_end.argtypes = [vp]
        L.sae_shard_set_avg_mode.argtypes = [vp, i32]
        L.sae_set_local_steps.argtypes = [vp, i32]
        L.sae_avg_due.argtypes = [vp]
        L.sae_num_padded.argtypes = [vp]
        L.sae_num_padded.restype = i64
        L.sae_avg_local_sum.argtypes = [vp, vp]
        L.sae_avg_set.argtypes = [vp, vp]
        L.sae_sign_compress_noalloc.argtypes = [vp, i64, vp, vp, vp, vp]
        L.sae_noalloc_max_elements.argtypes = []
        L.sae_noalloc_max_elements.restype = i64
        _lib = L
    return _lib


def _check(status, what, handle=None):
    if status != OK:
        raise SaeError(status, what, lib().sae_last_cuda_error(handle))


class Sae:
    """One Algorithm-1 run on one GPU.  Methods mirror the C entry points one to one.

    With `shard=(worker_begin, num_local_workers)` the handle is one shard of a run whose K = num_workers
    workers are spread over several handles (sae_init_shard): `step_begin` / `step_end` replace `step`,
    gradients are [num_local][d], and worker indices of the getters are local."""

    def __init__(self, num_workers, tensor_sizes, x0, compressor=SIGN, server_compress=1, mode=SAEF, avg_period=0,
                 momentum=0.9, weight_decay=0.0, topk_num=1, topk_den=100, device=None, stream=None, shard=None,
                 local_steps=1):
        import torch
        self.torch = torch
        if not (x0.is_cuda and x0.dtype == torch.float32 and x0.is_contiguous()):
            raise ValueError("x0 must be a contiguous float32 CUDA tensor")
        self.device = x0.device if device is None else torch.device(device)
        self.sizes = np.ascontiguousarray(tensor_sizes, dtype=np.int64)
        if x0.numel() != int(self.sizes.sum()):
            raise ValueError("x0 has the wrong length")
        self.K = int(num_workers)
        self.T = len(self.sizes)
        self.compressor = compressor
        self.keeps_momentum = not (momentum == 0.0 and avg_period != 1)     # mu = 0: m^(k) is not state
        self.stream = torch.cuda.current_stream(self.device).cuda_stream if stream is None else stream
        cfg = SaeConfig(ABI_VERSION, self.K, self.T, self.sizes.ctypes.data_as(C.POINTER(C.c_int64)), compressor,
                        server_compress, mode, avg_period, momentum, weight_decay, topk_num, topk_den,
                        self.device.index or 0, C.c_void_p(self.stream))
        h = C.c_void_p()
        self.shard = shard
        self.K_total = self.K
        if shard is None:
            _check(lib().sae_init(C.byref(cfg), x0.data_ptr(), C.byref(h)), "sae_init")
        else:
            _check(lib().sae_init_shard(C.byref(cfg), int(shard[0]), int(shard[1]), x0.data_ptr(), C.byref(h)),
                   "sae_init_shard")
            self.K = int(shard[1])          # rows held here: gradients are [K][d], getters take 0..K-1
        self.h = h
        if local_steps != 1:
            self.set_local_steps(local_steps)
        self.d = int(lib().sae_num_params(h))
        self.nwords = int(lib().sae_num_words(h))

    def set_local_steps(self, period):
        """sae_set_local_steps: the model differences are communicated every `period` iterations."""
        _check(lib().sae_set_local_steps(self.h, int(period)), "sae_set_local_steps", self.h)

    def close(self):
        if getattr(self, "h", None):
            lib().sae_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _vec(self, dtype=None, n=None):
        t = self.torch
        return t.empty(self.d if n is None else n, dtype=dtype or t.float32, device=self.device)

    def step(self, grads, lr):
        t = self.torch
        if not (grads.is_cuda and grads.dtype == t.float32 and grads.is_contiguous() and grads.numel() == self.K * self.d):
            raise ValueError("grads must be a contiguous float32 CUDA tensor of K*d elements")
        _check(lib().sae_step(self.h, grads.data_ptr(), lr), "sae_step", self.h)

    def shard_export(self):
        """Where this shard's message rows live, as SHARD_BLOB_BYTES bytes to hand to every shard."""
        buf = (C.c_ubyte * SHARD_BLOB_BYTES)()
        _check(lib().sae_shard_export(self.h, buf, SHARD_BLOB_BYTES), "sae_shard_export", self.h)
        return bytes(buf)

    def shard_attach(self, blob):
        buf = (C.c_ubyte * SHARD_BLOB_BYTES).from_buffer_copy(blob)
        _check(lib().sae_shard_attach(self.h, buf, SHARD_BLOB_BYTES), "sae_shard_attach", self.h)

    def shard_detach(self):
        _check(lib().sae_shard_detach(self.h), "sae_shard_detach", self.h)

    def step_begin(self, grads_local, lr):
        t = self.torch
        if not (grads_local.is_cuda and grads_local.dtype == t.float32 and grads_local.is_contiguous()
                and grads_local.numel() == self.K * self.d):
            raise ValueError("grads_local must be a contiguous float32 CUDA tensor of num_local*d elements")
        _check(lib().sae_step_begin(self.h, grads_local.data_ptr(), lr), "sae_step_begin", self.h)

    def step_end(self):
        _check(lib().sae_step_end(self.h), "sae_step_end", self.h)

    def shard_set_avg_mode(self, external_sum):
        _check(lib().sae_shard_set_avg_mode(self.h, 1 if external_sum else 0), "sae_shard_set_avg_mode", self.h)

    @property
    def avg_due(self):
        return bool(lib().sae_avg_due(self.h))

    def avg_local_sum(self, buf=None):
        """sum_k e^(k) over this shard's workers into buf (padded layout, sae_num_padded floats)."""
        if buf is None:
            buf = self._vec(n=int(lib().sae_num_padded(self.h)))
        _check(lib().sae_avg_local_sum(self.h, buf.data_ptr()), "sae_avg_local_sum", self.h)
        return buf

    def avg_set(self, buf):
        _check(lib().sae_avg_set(self.h, buf.data_ptr()), "sae_avg_set", self.h)

    def step_host(self, grads_host, lr):
        t = self.torch
        if grads_host.is_cuda or grads_host.dtype != t.float32 or not grads_host.is_contiguous() \
                or grads_host.numel() != self.K * self.d:
            raise ValueError("grads_host must be a contiguous float32 host tensor of K*d elements")
        _check(lib().sae_step_host(self.h, grads_host.data_ptr(), lr), "sae_step_host", self.h)

    def get_params(self, out=None):
        out = self._vec() if out is None else out
        _check(lib().sae_get_params(self.h, out.data_ptr()), "sae_get_params", self.h)
        return out

    def get_params_host(self, out_host):
        _check(lib().sae_get_params_host(self.h, out_host.data_ptr()), "sae_get_params_host", self.h)
        return out_host

    def get_step_ahead(self, worker, out=None):
        out = self._vec() if out is None else out
        _check(lib().sae_get_step_ahead(self.h, worker, out.data_ptr()), "sae_get_step_ahead", self.h)
        return out

    def get_state(self, which, worker=0):
        t = self.torch
        if which in (STATE_MOMENTUM, STATE_WORKER_ERROR, STATE_SERVER_ERROR):
            out = self._vec()
        elif which in (STATE_WORKER_SCALES, STATE_SERVER_SCALES):
            out = self._vec(n=self.T)
        elif which in (STATE_WORKER_TAU, STATE_SERVER_TAU):
            out = self._vec(dtype=t.int32, n=self.T)
        elif which == STATE_TOPK_FALLBACKS:
            out = self._vec(dtype=t.int32, n=2)
        else:
            out = self._vec(dtype=t.int32, n=self.nwords)
        _check(lib().sae_get_state(self.h, which, worker, out.data_ptr(), out.numel() * out.element_size()),
               "sae_get_state", self.h)
        return out

    def save_state(self):
        t = self.torch
        blob = t.empty(int(lib().sae_state_bytes(self.h)), dtype=t.uint8, device=self.device)
        _check(lib().sae_save_state(self.h, blob.data_ptr(), blob.numel()), "sae_save_state", self.h)
        return blob

    def load_state(self, blob):
        _check(lib().sae_load_state(self.h, blob.data_ptr(), blob.numel()), "sae_load_state", self.h)

    def get_mismatch(self):
        out = (C.c_double * 2)()
        _check(lib().sae_get_mismatch(self.h, out), "sae_get_mismatch", self.h)
        return float(out[0]), float(out[1])

    @property
    def iteration(self):
        return int(lib().sae_iteration(self.h))

    @property
    def kernel_launches(self):
        return int(lib().sae_kernel_launches(self.h))

    def sync(self):
        _check(lib().sae_sync(self.h), "sae_sync", self.h)

    def set_profiling(self, enabled):
        _check(lib().sae_set_profiling(self.h, 1 if enabled else 0), "sae_set_profiling", self.h)

    def get_kernel_times(self):
        ms = (C.c_float * NUM_KERNELS)()
        cnt = (C.c_int64 * NUM_KERNELS)()
        _check(lib().sae_get_kernel_times(self.h, ms, cnt), "sae_get_kernel_times", self.h)
        return {lib().sae_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(NUM_KERNELS)
                if cnt[i] > 0}


def noalloc_max_elements():
    return int(lib().sae_noalloc_max_elements())


def sign_compress_noalloc(v, words, scale, range_flag=None, stream=None):
    """Scaled-sign compressor of one tensor through `sae_sign_compress_noalloc`: for callers that cannot
    allocate device memory (they pass every buffer; the library's only scratch is a fixed array in its
    image).  v: float32 CUDA tensor (n elements); words: int32 CUDA tensor of ceil(n/32) elements; scale:
    float32 CUDA tensor of 1 element; range_flag: optional int32 CUDA tensor of 1 element.  Asynchronous on
    the current stream of v's device.  Calls must not overlap on the GPU (they share the scratch array)."""
    import torch
    n = v.numel()
    if not (v.is_cuda and v.dtype == torch.float32 and v.is_contiguous()):
        raise ValueError("v must be a contiguous float32 CUDA tensor")
    if words.numel() < (n + 31) // 32 or words.element_size() != 4 or not words.is_cuda or scale.numel() < 1:
        raise ValueError("output buffers are too small")
    with torch.cuda.device(v.device):
        st = torch.cuda.current_stream(v.device).cuda_stream if stream is None else stream
        rc = lib().sae_sign_compress_noalloc(v.data_ptr(), n, words.data_ptr(), scale.data_ptr(),
                                             range_flag.data_ptr() if range_flag is not None else None, C.c_void_p(st))
    _check(rc, "sae_sign_compress_noalloc")
