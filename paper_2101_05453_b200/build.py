"""Builds libqlstm.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libqlstm.so")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-diag-suppress", "550"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(INCLUDE, "*.h"))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = LIB + f".{os.getpid()}.tmp"
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources()
        subprocess.check_call(cmd)
        os.replace(tmp, LIB)
    return LIB


HOST_CHECK_SRC = os.path.join(CSRC, "host_check", "qmath_host.cpp")
HOST_CHECK_LIB = os.path.join(HERE, "libqmath_host.so")


def build_host_check(force: bool = False) -> str:
    """g++ build of the kernels' integer arithmetic (qmath.cuh) for CPU-side sweeps in the tests."""
    deps = [HOST_CHECK_SRC, os.path.join(CSRC, "qmath.cuh")]
    if force or not os.path.exists(HOST_CHECK_LIB) or any(os.path.getmtime(f) > os.path.getmtime(HOST_CHECK_LIB) for f in deps):
        tmp = HOST_CHECK_LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-o", tmp, HOST_CHECK_SRC])
        os.replace(tmp, HOST_CHECK_LIB)
    return HOST_CHECK_LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
