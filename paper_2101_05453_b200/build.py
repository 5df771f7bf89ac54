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
    """Compiles every .cu file to an object (in parallel: the kernel files take about a minute each) and links them."""
    if force or needs_build():
        from concurrent.futures import ThreadPoolExecutor
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        objdir = os.path.join(HERE, "_build", str(os.getpid()))
        os.makedirs(objdir, exist_ok=True)
        flags = [f for f in NVCC_FLAGS if f != "-shared"] + (["-Xptxas", "-v"] if verbose else [])

        def compile_one(src):
            obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
            subprocess.check_call([nvcc] + flags + ["-c", "-o", obj, src])
            return obj

        with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
            objs = list(pool.map(compile_one, sources()))
        tmp = LIB + f".{os.getpid()}.tmp"
        subprocess.check_call([nvcc, "-shared", "-Xcompiler", "-fPIC", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs)
        os.replace(tmp, LIB)
        for o in objs:
            os.unlink(o)
        os.rmdir(objdir)
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
