"""Builds libkvr.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
SO = os.path.join(PKG, "libkvr.so")
SOURCES = ["kvr_kernels.cu", "kvr_engine.cu", "kvr_lib.cu", "kvr_noalloc.cu", "kvr_policy.cpp", "kvr_controller.cpp", "kvr_numa.cpp"]
DEPS = SOURCES + ["kvr_kernels.cuh", "kvr_meta.hpp", "kvr_numa.hpp", "kvr_pool.hpp", os.path.join("..", "..", "include", "kvr.h")]


def stale():
    if not os.path.exists(SO):
        return True
    t = os.path.getmtime(SO)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force=False, verbose=False):
    """Compile when sources are newer than the library.  Returns the path of libkvr.so."""
    if not (force or stale()):
        return SO
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = SO + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-Wall", "-shared", "-cudart", "static",
           "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, SO)
    return SO


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
