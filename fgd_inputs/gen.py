"""Seeded synthetic inputs for the outer-round tests and benchmark (CPU side, numpy).

This module holds NO arithmetic of the method: it only manufactures input data
(initial parameters, per-round local drift standing in for the H inner steps, the
per-worker drift scales, a dense doubly-stochastic matrix) and is the one piece the
oracle-side tests and the CUDA-side tests may both use.

Every value is a pure function of (seed, tensor_id, round, worker m, column p), so
any column block of any round can be regenerated anywhere.  The generator uses only
integer operations plus IEEE-754 round-to-nearest fp32 multiplies/adds, so the CUDA
twin in ``gen.cu`` produces the SAME BITS:

    key  = mix64((mix64((mix64((mix64(seed + G) ^ tensor_id) + G) ^ round) + G) ^ m) + G)
    z_a  = mix64(key + (2p + 1) G),  z_b = mix64(key + (2p + 2) G)      (mod 2^64)
    S    = sum of the eight 16-bit fields of z_a and z_b                 (0 .. 524280)
    eps  = fp32(S - 262140) * fp32(1 / sqrt(8 (2^32 - 1) / 12))          (one rounding)

eps is an Irwin-Hall(8) variate scaled to zero mean and unit variance (support
+-4.9 sigma), the stand-in for a standard normal.  mix64 is the splitmix64 finaliser,
G = 0x9E3779B97F4A7C15.
"""
from __future__ import annotations

import math

import numpy as np

G = np.uint64(0x9E3779B97F4A7C15)
_G_INT = 0x9E3779B97F4A7C15
_MASK = (1 << 64) - 1

TENSOR_THETA0 = 1       # initial parameters shared by all workers
TENSOR_DRIFT = 2        # per-round, per-worker local drift
TENSOR_SIGMA = 3        # per-worker drift scale
TENSOR_WORKER_OFFSET = 4  # optional per-worker offset of the initial parameters
TENSOR_DENSE_W = 5      # dense mixing matrix seed values
TENSOR_MOMENTUM = 6     # optional non-zero initial momentum (tests only)
TENSOR_AUX = 7          # any other test tensor

IH_MEAN = 262140                                  # 4 * 65535
IH_INV_STD = np.float32(1.0 / math.sqrt(8.0 * (2.0 ** 32 - 1.0) / 12.0))


def _mix64_int(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def row_key(seed: int, tensor_id: int, rnd: int, m: int) -> int:
    k = _mix64_int(seed + _G_INT)
    for x in (tensor_id, rnd, m):
        k = _mix64_int(((k ^ (x & _MASK)) + _G_INT) & _MASK)
    return k


def _mix64(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def _sum16(z: np.ndarray) -> np.ndarray:
    m = np.uint64(0xFFFF)
    return ((z & m) + ((z >> np.uint64(16)) & m) + ((z >> np.uint64(32)) & m)
            + (z >> np.uint64(48))).astype(np.int64)


def std_normal(seed: int, tensor_id: int, rnd: int, m: int, p0: int, p1: int) -> np.ndarray:
    """eps[p] for columns p0 <= p < p1 of row m, float32."""
    with np.errstate(over="ignore"):
        key = np.uint64(row_key(seed, tensor_id, rnd, m))
        p = np.arange(p0, p1, dtype=np.uint64)
        za = _mix64(key + (np.uint64(2) * p + np.uint64(1)) * G)
        zb = _mix64(key + (np.uint64(2) * p + np.uint64(2)) * G)
    c = (_sum16(za) + _sum16(zb) - IH_MEAN).astype(np.float32)   # exact: |c| < 2^24
    return c * IH_INV_STD


def uniform01(seed: int, tensor_id: int, rnd: int, m: int, p: int) -> float:
    """One double in [0, 1) with 53 random bits, from the same key schedule."""
    z = _mix64_int(row_key(seed, tensor_id, rnd, m) + (2 * p + 1) * _G_INT)
    return (z >> 11) / float(1 << 53)


def scaled_normal(seed, tensor_id, rnd, K, P, scales, p0=0, p1=None) -> np.ndarray:
    """[K, p1-p0] float32 with row m = fp32(scales[m]) * eps (one rounding per element)."""
    p1 = P if p1 is None else p1
    scales = np.broadcast_to(np.asarray(scales, dtype=np.float32), (K,))
    out = np.empty((K, p1 - p0), dtype=np.float32)
    for m in range(K):
        out[m] = scales[m] * std_normal(seed, tensor_id, rnd, m, p0, p1)
    return out


def theta0(seed: int, K: int, P: int, std: float = 0.02, worker_std: float = 0.0,
           p0: int = 0, p1=None) -> np.ndarray:
    """Initial outer parameters [K, p1-p0]: one N(0, std^2)-like draw shared by all workers
    ("all workers start identical"), plus an optional per-worker offset of scale worker_std
    (used by the parity variant that makes Mix1 non-trivial in a single round)."""
    p1 = P if p1 is None else p1
    base = np.float32(std) * std_normal(seed, TENSOR_THETA0, 0, 0, p0, p1)
    out = np.repeat(base[None, :], K, axis=0)
    if worker_std > 0.0:
        out = out + scaled_normal(seed, TENSOR_WORKER_OFFSET, 0, K, P, worker_std, p0, p1)
    return np.ascontiguousarray(out, dtype=np.float32)


def drift_sigmas(seed: int, K: int, lo: float, hi: float) -> np.ndarray:
    """Per-worker drift scale sigma_m ~ U[lo, hi), drawn once from the seed, float32."""
    return np.array([lo + (hi - lo) * uniform01(seed, TENSOR_SIGMA, 0, m, 0) for m in range(K)],
                    dtype=np.float32)


def local_params(theta_prev: np.ndarray, sigmas, seed: int, rnd: int, p0: int = 0) -> np.ndarray:
    """Stand-in for the H inner steps: theta_local = theta_prev + fp32(sigma_m * eps).

    ``theta_prev`` is the [K, n] float32 block starting at column p0.  Two fp32 roundings
    (multiply, then add), exactly as the CUDA twin does.
    """
    theta_prev = np.asarray(theta_prev, dtype=np.float32)
    K, n = theta_prev.shape
    drift = scaled_normal(seed, TENSOR_DRIFT, rnd, K, p0 + n, sigmas, p0, p0 + n)
    return theta_prev + drift


def sinkhorn_W(seed: int, K: int, iters: int = 1000, tol: float = 1e-14) -> np.ndarray:
    """Dense symmetric doubly-stochastic [K, K] matrix, returned as float32.

    U ~ Uniform[0.1, 1) from the seed, A = (U + U^T)/2, alternate row / column
    normalisation in float64 until every row and column sum is within ``tol`` of 1,
    symmetrise once more, round to fp32 once.  The fp32 values ARE the input: both the
    oracle and the CUDA path consume them as given.
    """
    U = np.array([[0.1 + 0.9 * uniform01(seed, TENSOR_DENSE_W, 0, i, j) for j in range(K)]
                  for i in range(K)], dtype=np.float64)
    A = 0.5 * (U + U.T)
    for _ in range(iters):
        A = A / A.sum(axis=1, keepdims=True)
        A = A / A.sum(axis=0, keepdims=True)
        if (np.abs(A.sum(axis=1) - 1.0).max() < tol and np.abs(A.sum(axis=0) - 1.0).max() < tol):
            break
    A = 0.5 * (A + A.T)
    return np.ascontiguousarray(A, dtype=np.float32)
