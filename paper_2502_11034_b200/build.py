"""Build step: compile csrc/adagc.cu (one translation unit; it includes the other files of csrc/) into libadagc.so
(next to this file) for sm_100a."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_HERE, "csrc", "adagc.cu")
HEADER = os.path.join(os.path.dirname(_HERE), "include", "adagc.h")
LIB = os.path.join(_HERE, "libadagc.so")

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-shared", "-Xcompiler", "-fPIC"]


def nvcc_path() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


LIB_CHECKED = os.path.join(_HERE, "libadagc_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the CUDA library if it is missing or older than its sources; returns its path.
    checked: the debugging build (-DADAGC_BOUNDS_CHECK, libadagc_checked.so) whose kernels verify every chunk-table entry
    before they use it; select it at run time with ADAGC_LIBRARY=<path>."""
    lib = LIB_CHECKED if checked else LIB
    csrc = os.path.dirname(SRC)
    newest = max([os.path.getmtime(HEADER)] + [os.path.getmtime(os.path.join(csrc, f)) for f in os.listdir(csrc)])
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= newest:
        return lib
    cmd = ([nvcc_path()] + NVCC_FLAGS + (["-DADAGC_BOUNDS_CHECK"] if checked else []) +
           (["-Xptxas", "-v"] if verbose else []) + ["-o", lib, SRC])
    subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose=True, checked="--checked" in sys.argv))
