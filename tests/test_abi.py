"""The C-ABI library loads without a GPU and exports every function include/sae.h declares; host-side
argument checks answer with status codes (no compute is attempted here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2008_05823_b200 import binding as sb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sae.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(sae_[a-z_]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_function():
    L = sb.lib()
    names = declared_functions()
    assert len(names) >= 15
    for name in names:
        assert hasattr(L, name), f"{name} is declared in sae.h but not exported by libsae.so"
    assert sorted(sb.EXPORTS) == names


def test_strerror_and_kernel_names():
    L = sb.lib()
    assert L.sae_strerror(0) == b"ok"
    assert b"invalid" in L.sae_strerror(sb.ERR_INVALID_ARG)
    assert L.sae_kernel_name(0) == b"worker_pass"
    assert L.sae_kernel_name(99) == b""


def test_host_side_argument_checks_need_no_gpu():
    L = sb.lib()
    sizes = np.array([8, 8], dtype=np.int64)
    h = C.c_void_p()

    def cfg(**kw):
        base = dict(abi_version=sb.ABI_VERSION, num_workers=2, num_tensors=2,
                    tensor_sizes=sizes.ctypes.data_as(C.POINTER(C.c_int64)), compressor=sb.SIGN, server_compress=1,
                    mode=sb.SAEF, avg_period=0, momentum=0.9, weight_decay=0.0, topk_num=1, topk_den=100, device=0,
                    stream=None)
        base.update(kw)
        return sb.SaeConfig(**base)

    fake_x0 = C.c_void_p(16)         # never dereferenced: the checks below fail first
    assert L.sae_init(None, fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(abi_version=99)), fake_x0, C.byref(h)) == sb.ERR_ABI
    assert L.sae_init(C.byref(cfg(num_workers=0)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(num_workers=5000)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(momentum=1.0)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(weight_decay=-1.0)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(compressor=3)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(compressor=sb.TOPK, topk_den=0)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_init(C.byref(cfg(avg_period=-1)), fake_x0, C.byref(h)) == sb.ERR_INVALID_ARG
    bad = np.array([8, 0], dtype=np.int64)
    assert L.sae_init(C.byref(cfg(tensor_sizes=bad.ctypes.data_as(C.POINTER(C.c_int64)))), fake_x0,
                      C.byref(h)) == sb.ERR_INVALID_ARG
    assert L.sae_step(None, fake_x0, 0.1) == sb.ERR_INVALID_ARG
    assert L.sae_sync(None) == sb.ERR_INVALID_ARG
    assert L.sae_iteration(None) == -1
    L.sae_destroy(None)


def test_init_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    L = sb.lib()
    sizes = np.array([8], dtype=np.int64)
    cfg = sb.SaeConfig(sb.ABI_VERSION, 1, 1, sizes.ctypes.data_as(C.POINTER(C.c_int64)), sb.SIGN, 1, sb.SAEF, 0, 0.9,
                       0.0, 1, 100, 0, None)
    h = C.c_void_p()
    assert L.sae_init(C.byref(cfg), C.c_void_p(16), C.byref(h)) == sb.ERR_CUDA
    assert not h.value
    assert L.sae_last_cuda_error(None) != 0
