"""Builds librobe.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "librobe.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh"))
    deps.append(os.path.join(_HERE, "..", "include", "robe.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + sources()
        subprocess.run(cmd, check=True)
    return LIB


DEBUG_LIB = os.path.join(_HERE, "librobe_debug.so")


def build_debug(force: bool = False) -> str:
    """The index-check build: the same sources with -DROBE_DEBUG, compiled as ONE translation unit
    (a generated file that includes every .cu) so that the device word the checks report into
    exists once."""
    stale = not os.path.exists(DEBUG_LIB) or (os.path.exists(LIB) and os.path.getmtime(DEBUG_LIB) < os.path.getmtime(LIB))
    if force or stale or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        unity = os.path.join(CSRC, "_unity_debug.cu")
        try:
            with open(unity, "w") as f:
                for src in sources():
                    if os.path.basename(src) != "_unity_debug.cu":
                        f.write(f'#include "{os.path.basename(src)}"\n')
            subprocess.run([nvcc] + NVCC_FLAGS + ["-DROBE_DEBUG", "-o", DEBUG_LIB, unity], check=True)
        finally:
            if os.path.exists(unity):
                os.unlink(unity)
    return DEBUG_LIB


if __name__ == "__main__":
    build(force=True, verbose="-v" in sys.argv)
    print(LIB)
    if "--debug" in sys.argv:
        print(build_debug(force=True))
