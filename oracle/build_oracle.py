"""Builds the CPU oracle (test infrastructure) into oracle/libsae_oracle.so with g++.

-ffp-contract=off keeps every floating-point operation separately rounded except the explicit fma calls;
-mfma lets std::fma compile to the hardware instruction (same result as the library routine, faster).
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sae_oracle.cpp")
OUT = os.path.join(HERE, "libsae_oracle.so")


def build(force: bool = False) -> str:
    if not force and os.path.exists(OUT) and os.path.getmtime(OUT) >= os.path.getmtime(SRC):
        return OUT
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-mavx2", "-mfma", "-fopenmp", "-fPIC", "-shared",
           "-Wall", "-o", OUT, SRC]
    subprocess.check_call(cmd)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
