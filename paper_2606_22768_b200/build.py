"""Build ``libfgd.so`` (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Run as ``python paper_2606_22768_b200/build.py`` (as a script: importing the package needs the
library to exist already).  Needs only nvcc (cross-compiles without
a GPU).  The library links the CUDA runtime statically, so it loads on machines without a
driver; only the GPU entry points then fail (with FGD_ERR_CUDA).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OUT = os.path.join(HERE, "libfgd.so")
SOURCES = ["fgd_api.cu", "fgd_noalloc.cu", "fgd_host.cpp"]
HEADERS = ["fgd_kernels.cuh", "fgd_step_tma.cuh", "fgd_internal.h", os.path.join(ROOT, "include", "fgd.h")]

NVCC_FLAGS = ["-std=c++20", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-I" + os.path.join(ROOT, "include")]


def stale() -> bool:
    if not os.path.exists(OUT):
        return True
    t = os.path.getmtime(OUT)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [h if os.path.isabs(h) else os.path.join(CSRC, h) for h in HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        cmd = ["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", OUT] + \
              [os.path.join(CSRC, s) for s in SOURCES]
        subprocess.run(cmd, check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
