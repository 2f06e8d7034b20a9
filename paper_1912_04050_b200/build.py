"""Build ``libbenes.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB = os.path.join(_HERE, "libbenes.so")
LIB_DEBUG = os.path.join(_HERE, "libbenes_debug.so")      # the same sources with -DBENES_DEBUG (index guards report)

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every kernel for sm_100a; returns the path of the shared library
    (debug=True: the checked build, libbenes_debug.so)."""
    lib = LIB_DEBUG if debug else LIB
    if force or _stale(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = lib + ".%d.tmp" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-DBENES_DEBUG"] if debug else []) + \
              (["-Xptxas", "-v"] if verbose else []) + ["-I", INCLUDE, "-I", CSRC, "-o", tmp] + sources()
        subprocess.check_call(cmd)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose=True))
