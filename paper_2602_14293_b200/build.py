"""Build the CUDA library (libfc.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libfc.so")
LIB_DEBUG = os.path.join(PKG, "libfc_debug.so")   # the same sources with -DFC_DEBUG: address checks in the kernels (see include/fc.h)


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile the library (debug=True: the bounds-checked variant, libfc_debug.so) unless it is up to date."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not needs_build(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "--threads", "0",   # the source files are compiled side by side (the elementwise kernels alone take two minutes)
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "-o", lib] + sources()
    if debug:
        cmd.insert(1, "-DFC_DEBUG")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    for d in os.environ.get("FC_DEFINES", "").split():   # development builds: e.g. FC_DEFINES="FC_PROF"
        cmd.insert(1, "-D" + d)
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
