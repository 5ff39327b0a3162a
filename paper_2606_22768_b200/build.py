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
SOURCES = ["fgd_api.cu", "fgd_step_tma.cu", "fgd_step_tma_g0.cu", "fgd_step_tma_g1.cu", "fgd_step_tma_g2.cu", "fgd_step_tma_g3.cu",
           "fgd_step_reg.cu", "fgd_step_rows.cu", "fgd_mix_gather_tma.cu", "fgd_noalloc.cu", "fgd_js.cu", "fgd_pattern_probe.cu", "fgd_from_host.cu", "fgd_host.cpp"]
HEADERS = ["fgd_kernels.cuh", "fgd_step_tma.cuh", "fgd_step_dense_tc.cuh", "fgd_mix_dense_tc.cuh", "fgd_step_gossip_tc.cuh", "fgd_step_tma.h", "fgd_tma_host.h", "fgd_step_tma_launch.inl", "fgd_ctx.h", "fgd_internal.h", "fgd_nvtx.h", os.path.join(ROOT, "include", "fgd.h")]

NVCC_FLAGS = ["-std=c++20", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I" + os.path.join(ROOT, "include")]
OBJ_DIR = os.path.join(HERE, "build")


def stale() -> bool:
    if not os.path.exists(OUT):
        return True
    t = os.path.getmtime(OUT)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + [h if os.path.isabs(h) else os.path.join(CSRC, h) for h in HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        from concurrent.futures import ThreadPoolExecutor
        os.makedirs(OBJ_DIR, exist_ok=True)
        extra = ["-Xptxas", "-v"] if verbose else []

        def compile_one(src):
            obj = os.path.join(OBJ_DIR, os.path.splitext(src)[0] + ".o")
            subprocess.run(["nvcc"] + NVCC_FLAGS + extra + ["-c", "-o", obj, os.path.join(CSRC, src)], check=True)
            return obj

        with ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:   # one nvcc per translation unit
            objs = list(pool.map(compile_one, SOURCES))
        subprocess.run(["nvcc", "-shared", "-o", OUT] + objs + ["-ldl"], check=True)
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
