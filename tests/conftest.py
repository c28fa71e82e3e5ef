import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200 with -m gpu)")
    # A fresh checkout has no built libraries (they are not in the history): build what is missing, once,
    # so that the suite does not depend on a build step having run before it.  nvcc cross-compiles without a GPU.
    from paper_2008_05823_b200 import build as cuda_build
    if not all(os.path.exists(os.path.join(cuda_build.HERE, name)) for name in cuda_build.TARGETS):
        cuda_build.build()


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def free_port():
    """A TCP port nobody listens on right now (the rendezvous of the child processes)."""
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return str(s.getsockname()[1])
