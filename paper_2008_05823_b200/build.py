"""Builds the CUDA libraries in-tree for sm_100a with nvcc:

  libsae.so        -- the C-ABI library declared in include/sae.h
  libsae_synth.so  -- the seeded synthetic-gradient generator used by tests and the benchmark

Usage: python -m paper_2008_05823_b200.build [--force] [--verbose]
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
              "-Xcompiler", "-fPIC", "-shared"]

TARGETS = {
    "libsae.so": (["sae.cu", "sae_noalloc.cu"], ["sae_kernels.cuh", "sae_worker_tma.cuh", "sae_worker_fused.cuh", "sae_worker_small.cuh", "sae_topk.cuh", "sae_shard_topk.cuh", "sae_device.cuh", os.path.join(INCLUDE, "sae.h")]),
    "libsae_synth.so": (["synth_gen.cu"], []),
}


def _stale(out, deps):
    if not os.path.exists(out):
        return True
    t = os.path.getmtime(out)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False):
    nvcc = os.environ.get("NVCC", "nvcc")
    outs = []
    for name, (srcs, hdrs) in TARGETS.items():
        out = os.path.join(HERE, name)
        src_paths = [os.path.join(CSRC, s) for s in srcs]
        dep_paths = src_paths + [h if os.path.isabs(h) else os.path.join(CSRC, h) for h in hdrs]
        if force or _stale(out, dep_paths):
            extra = os.environ.get("SAE_NVCC_EXTRA", "").split()
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", out] + src_paths
            subprocess.check_call(cmd)
        outs.append(out)
    return outs


if __name__ == "__main__":
    for o in build(force="--force" in sys.argv, verbose="--verbose" in sys.argv):
        print(o)
