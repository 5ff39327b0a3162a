"""CUDA twin of ``gen`` (same bits, produced directly in HBM) -- input manufacture only.

``local_steps`` doubles as the stand-in compute kernel that models the H inner training
steps between two outer rounds.  Built in-tree by ``build()`` into ``libfgd_inputs.so``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import gen

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.cu")
LIB_PATH = os.path.join(_HERE, "libfgd_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB_PATH) or os.path.getmtime(LIB_PATH) < os.path.getmtime(_SRC):
        subprocess.run(["nvcc", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
                        "-Xcompiler", "-fPIC", "-shared", "-o", LIB_PATH, _SRC], check=True)
    return LIB_PATH


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run fgd_inputs.gpu.build()")
        lib = ctypes.CDLL(LIB_PATH)
        lib.fgdin_fill.restype = ctypes.c_int
        lib.fgdin_fill.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64,
                                   ctypes.c_int64, ctypes.c_uint64, ctypes.c_int, ctypes.c_int64,
                                   ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                   ctypes.c_void_p]
        _lib = lib
    return _lib


def _fill(out, base, seed, tensor_id, rnd, scales, shared_row, add, stream=None):
    import torch
    K, P = out.shape
    assert out.is_cuda and out.dtype == torch.float32 and out.stride(1) == 1
    ld = out.stride(0) if K > 1 else P
    scales = np.ascontiguousarray(np.broadcast_to(np.asarray(scales, dtype=np.float32), (K,)))
    st = torch.cuda.current_stream().cuda_stream if stream is None else getattr(stream, "cuda_stream", stream)
    rc = _load().fgdin_fill(out.data_ptr(), None if base is None else base.data_ptr(), K, P, ld, seed,
                            tensor_id, rnd, scales.ctypes.data, int(shared_row), int(add),
                            float(gen.IH_INV_STD), st)
    if rc != 0:
        raise RuntimeError(f"fgdin_fill failed with code {rc}")


def theta0(out, seed: int, std: float = 0.02, worker_std: float = 0.0):
    """Fill ``out`` [K, P] like ``gen.theta0`` (same bits)."""
    _fill(out, None, seed, gen.TENSOR_THETA0, 0, std, True, False)
    if worker_std > 0.0:
        _fill(out, out, seed, gen.TENSOR_WORKER_OFFSET, 0, worker_std, False, True)
    return out


def local_steps(theta_local, theta_prev, sigmas, seed: int, rnd: int, stream=None):
    """theta_local = theta_prev + fp32(sigma_m * eps(seed, round, m, p)) (same bits as gen.local_params)."""
    _fill(theta_local, theta_prev, seed, gen.TENSOR_DRIFT, rnd, sigmas, False, True, stream)
    return theta_local


def scaled_normal(out, seed: int, tensor_id: int, rnd: int, scales):
    _fill(out, None, seed, tensor_id, rnd, scales, False, False)
    return out
