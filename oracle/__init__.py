"""Float64 CPU oracle of the Factored Gossip DiLoCo outer round.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; never by the CUDA package.  The arithmetic lives in
``fgd_oracle.c`` (plain C loops, one per equation); this module compiles it with gcc,
loads it through ctypes, widens fp32 inputs to float64 (exact) and keeps the
multi-round state.  ``topology.py`` holds the oracle's own mixing-matrix builders.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import topology  # noqa: F401  (re-exported)

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fgd_oracle.c")
_LIB = os.path.join(_HERE, "libfgd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (-O2, no fast-math, OpenMP) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        lib.fgdo_num_threads.restype = ctypes.c_int
        lib.fgdo_set_num_threads.argtypes = [ctypes.c_int]
        lib.fgdo_outer_grad.argtypes = [ctypes.c_int, i64, dp, dp, dp]
        lib.fgdo_outer_grad.restype = None
        lib.fgdo_mix.argtypes = [ctypes.c_int, i64, dp, dp, dp]
        lib.fgdo_mix.restype = None
        lib.fgdo_nesterov.argtypes = [ctypes.c_int, i64, dp, dp, dp, ctypes.c_double,
                                      ctypes.c_double, dp]
        lib.fgdo_nesterov.restype = None
        lib.fgdo_round.argtypes = [ctypes.c_int, i64, dp, dp, dp, dp, dp, ctypes.c_double,
                                   ctypes.c_double, dp, dp, dp]
        lib.fgdo_round.restype = ctypes.c_int
        lib.fgdo_consensus_sumsq.argtypes = [ctypes.c_int, i64, dp, dp]
        lib.fgdo_consensus_sumsq.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().fgdo_num_threads())


def set_num_threads(n: int) -> None:
    _load().fgdo_set_num_threads(int(n))


def _f64(a) -> np.ndarray:
    """Widen to a C-contiguous float64 [K, P] array (exact for fp32 inputs)."""
    a = np.ascontiguousarray(np.asarray(a), dtype=np.float64)
    if a.ndim != 2:
        raise ValueError("expected a [K, P] array")
    return a


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _mat(W, K: int) -> np.ndarray:
    W = np.ascontiguousarray(np.asarray(W, dtype=np.float64))
    if W.shape != (K, K):
        raise ValueError(f"mixing matrix must be [{K}, {K}], got {W.shape}")
    return W


def outer_grad(theta_prev, theta_local) -> np.ndarray:
    """g = theta_prev - theta_local (the negated outer pseudo-gradient Delta)."""
    tp, tl = _f64(theta_prev), _f64(theta_local)
    g = np.empty_like(tp)
    _load().fgdo_outer_grad(tp.shape[0], tp.shape[1], _ptr(tp), _ptr(tl), _ptr(g))
    return g


def mix(W, v) -> np.ndarray:
    """Mix_W(v)_m = sum_n W[m][n] v_n, rows of ``v`` are workers."""
    v = _f64(v)
    W = _mat(W, v.shape[0])
    out = np.empty_like(v)
    _load().fgdo_mix(v.shape[0], v.shape[1], _ptr(W), _ptr(v), _ptr(out))
    return out


def nesterov(x, ghat, v, gamma: float, mu: float):
    """v' = mu v + ghat; theta_new = x - gamma (ghat + mu v').  Returns (theta_new, v')."""
    x, ghat = _f64(x), _f64(ghat)
    v = _f64(v).copy()
    out = np.empty_like(x)
    _load().fgdo_nesterov(x.shape[0], x.shape[1], _ptr(x), _ptr(ghat), _ptr(v), float(gamma),
                          float(mu), _ptr(out))
    return out, v


def outer_round(W1, W2, theta_prev, theta_local, v, gamma: float = 0.7, mu: float = 0.9,
                want_intermediates: bool = False):
    """One outer round.  Returns (theta_new, v_new) or (theta_new, v_new, x, ghat)."""
    tp, tl = _f64(theta_prev), _f64(theta_local)
    K, P = tp.shape
    W1, W2 = _mat(W1, K), _mat(W2, K)
    v = _f64(v).copy()
    out = np.empty_like(tp)
    x = np.empty_like(tp) if want_intermediates else None
    gh = np.empty_like(tp) if want_intermediates else None
    rc = _load().fgdo_round(K, P, _ptr(W1), _ptr(W2), _ptr(tp), _ptr(tl), _ptr(v), float(gamma),
                            float(mu), _ptr(out), _ptr(x) if x is not None else None,
                            _ptr(gh) if gh is not None else None)
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return (out, v, x, gh) if want_intermediates else (out, v)


def outer_round_ex(W1, W2, theta_prev, theta_local, v, gamma: float = 0.7, mu: float = 0.9,
                   mix2_ranges=None, average_momentum: bool = False):
    """One outer round of the two variants the paper adds on top of Algorithm 1, composed from
    the same one-equation primitives in the paper's order.

    mix2_ranges: list of (lo, hi) column ranges.  Mix2 is applied only to columns inside a range
        (the "-subset" configurations: Mix2 on a chosen subset of parameter blocks, "the rest pass
        through identity", App. A); None = every column.
    average_momentum: the GlobalM1S variants (App. B): Mix1 "also includes outer optimizer
        state", i.e. v_m <- Mix1(v)_m before the Nesterov update.
    Returns (theta_new, v_new).
    """
    tp, tl = _f64(theta_prev), _f64(theta_local)
    K, P = tp.shape
    x = mix(W1, tp)
    g = outer_grad(tp, tl)
    ghat = mix(W2, g)
    if mix2_ranges is not None:
        inside = np.zeros(P, dtype=bool)
        for lo, hi in mix2_ranges:
            inside[int(lo):int(hi)] = True
        ghat[:, ~inside] = g[:, ~inside]
    v_in = mix(W1, v) if average_momentum else _f64(v)
    return nesterov(x, ghat, v_in, gamma, mu)


def consensus_sumsq(theta) -> np.ndarray:
    """s[m] = sum_p (theta[m][p] - mean_p)^2."""
    th = _f64(theta)
    s = np.empty(th.shape[0], dtype=np.float64)
    if _load().fgdo_consensus_sumsq(th.shape[0], th.shape[1], _ptr(th), _ptr(s)) != 0:
        raise MemoryError("oracle scratch allocation failed")
    return s


def cd_finalize(s):
    """(CD_norm, CD_sq): the main-text definition (mean of norms) and the appendix one
    (mean of squared norms) of the L2 consensus distance."""
    s = np.asarray(s, dtype=np.float64)
    return float(np.mean(np.sqrt(s))), float(np.mean(s))


# ---------------------------------------------------------------- mixing matrices
def dense_W(kind: str, K: int, *, nbr=None, w=None, w_self=None, mask=None,
            renorm: int = topology.RENORM_NONE, W=None) -> np.ndarray:
    """Dense float64 row-convention matrix of a mix description.

    kind: "identity" | "mean" | "sparse" (nbr/w/w_self [+ mask + renorm]) | "dense" (W given).
    Global averaging ignores any mask: the paper's all-reduce restarts until it succeeds.
    """
    if kind == "identity":
        return np.array(topology.identity_matrix(K), dtype=np.float64)
    if kind == "mean":
        return np.array(topology.mean_matrix(K), dtype=np.float64)
    if kind == "sparse":
        nbr_l = [[int(n) for n in row] for row in np.asarray(nbr).tolist()]
        w_l = np.asarray(w, dtype=np.float64).tolist()
        ws_l = np.asarray(w_self, dtype=np.float64).tolist()
        mask_l = None if mask is None else np.asarray(mask).tolist()
        w_eff, ws_eff = topology.effective_weights(nbr_l, w_l, ws_l, mask_l, renorm)
        return np.array(topology.dense_from_sparse(nbr_l, w_eff, ws_eff), dtype=np.float64)
    if kind == "dense":
        return _mat(W, K)
    raise ValueError(f"unknown mix kind {kind!r}")
