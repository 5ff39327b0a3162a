"""B200-native Factored Gossip DiLoCo outer round: thin ctypes binding of ``libfgd.so``.

Argument marshalling only -- every step of the round runs in the library's CUDA kernels.
PyTorch is used by callers for device memory and streams; this module only reads
``data_ptr()`` / ``cuda_stream`` from what it is given.  There is no CPU fallback: importing
works anywhere (the host helpers are pure CPU), but the shared library must exist, and
every GPU entry point fails loudly when there is no CUDA device.

Entry points carry the C names (``fgd_outer_grad``, ``fgd_mix``, ``fgd_outer_step``,
``fgd_consensus_distance`` and the host helpers); see ``include/fgd.h`` for the contract.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfgd.so")

FGD_MAX_K = 64
FGD_MAX_D = 8

FGD_OK = 0
FGD_ERR_INVALID_ARG = -1
FGD_ERR_ALIGNMENT = -2
FGD_ERR_ALIAS = -3
FGD_ERR_UNSUPPORTED = -4
FGD_ERR_CUDA = -5
FGD_ERR_TIMEOUT = -6

FGD_MIX_IDENTITY, FGD_MIX_MEAN, FGD_MIX_SPARSE, FGD_MIX_DENSE = 0, 1, 2, 3
FGD_RENORM_NONE, FGD_RENORM_SELF_ABSORB, FGD_RENORM_METROPOLIS = 0, 1, 2
FGD_PATH_AUTO, FGD_PATH_REGISTER, FGD_PATH_TMA, FGD_PATH_TMA_FP32 = 0, 1, 2, 3


class FgdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"fgd status {status}: {message}")
        self.status = status
        self.message = message


class _CMixDesc(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("K", ctypes.c_int32), ("D", ctypes.c_int32),
                ("renorm", ctypes.c_int32), ("nbr", ctypes.c_void_p), ("w", ctypes.c_void_p),
                ("w_self", ctypes.c_void_p), ("edge_mask", ctypes.c_void_p), ("W", ctypes.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python paper_2606_22768_b200/build.py` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64, dbl = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
    descp = ctypes.POINTER(_CMixDesc)
    sig = {
        "fgd_create": (i32, [ctypes.POINTER(vp), i32, i32, i64, i64]),
        "fgd_destroy": (i32, [vp]),
        "fgd_last_error": (ctypes.c_char_p, [vp]),
        "fgd_status_string": (ctypes.c_char_p, [i32]),
        "fgd_launch_count": (i64, [vp]),
        "fgd_set_path": (i32, [vp, i32]),
        "fgd_device_status": (i32, [vp, vp]),
        "fgd_debug_set": (i32, [vp, i32, i64]),
        "fgd_debug_stream_pattern": (i32, [vp, vp, vp, vp, vp, vp]),
        "fgd_outer_grad": (i32, [vp, vp, vp, vp, vp]),
        "fgd_mix": (i32, [vp, descp, vp, vp, i32, vp]),
        "fgd_outer_step": (i32, [vp, descp, descp, vp, i32, vp, vp, vp, vp, dbl, dbl, vp, vp]),
        "fgd_outer_step_ex": (i32, [vp, descp, descp, vp, i32, vp, vp, vp, vp, dbl, dbl, vp, vp, vp]),
        "fgd_outer_step_from_host": (i32, [vp, descp, descp, vp, i32, vp, vp, vp, vp, vp, dbl, dbl, vp, i32, vp]),
        "fgd_consensus_distance": (i32, [vp, vp, vp, vp]),
        "fgd_consensus_distance_noalloc": (i32, [i32, i32, i64, i64, vp, vp, vp]),
        "fgd_js_distance": (i32, [i32, i32, i64, i64, i32, vp, vp, vp, vp, vp, vp]),
        "fgd_topo_ring": (i32, [i32, vp, vp, vp]),
        "fgd_topo_onepeer_xor": (i32, [i32, i64, vp, vp, vp]),
        "fgd_topo_hypercube": (i32, [i32, vp, vp, vp]),
        "fgd_topo_random_matching": (i32, [i32, u64, i64, i32, vp, vp, vp]),
        "fgd_edge_mask": (i32, [u64, i64, i32, dbl, i32, i32, vp, vp]),
        "fgd_hash64": (u64, [u64, u64, u64, u64, u64]),
        "fgd_effective_weights": (i32, [descp, vp, vp]),
        "fgd_dense_matrix": (i32, [descp, vp]),
        "fgd_cd_finalize": (i32, [vp, i32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib, tuple(sig)


_lib, EXPORTED_SYMBOLS = _load()


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


@dataclass
class MixDesc:
    """Host-side description of one mixing operator (mirrors ``fgd_mix_desc``)."""
    kind: int
    K: int
    D: int = 0
    renorm: int = FGD_RENORM_NONE
    nbr: Optional[np.ndarray] = None        # int32 [K, D]
    w: Optional[np.ndarray] = None          # float32 [K, D]
    w_self: Optional[np.ndarray] = None     # float32 [K]
    edge_mask: Optional[np.ndarray] = None  # uint8 [K, D]
    W: Optional[np.ndarray] = None          # float32 [K, K]
    _c: Optional[_CMixDesc] = field(default=None, repr=False, compare=False)

    def c(self) -> _CMixDesc:
        conv = lambda a, dt: None if a is None else np.ascontiguousarray(a, dtype=dt)
        self.nbr, self.w = conv(self.nbr, np.int32), conv(self.w, np.float32)
        self.w_self, self.edge_mask = conv(self.w_self, np.float32), conv(self.edge_mask, np.uint8)
        self.W = conv(self.W, np.float32)
        self._c = _CMixDesc(self.kind, self.K, self.D, self.renorm, _np_ptr(self.nbr), _np_ptr(self.w),
                            _np_ptr(self.w_self), _np_ptr(self.edge_mask), _np_ptr(self.W))
        return self._c

    # -- constructors -----------------------------------------------------------------
    @staticmethod
    def identity(K: int) -> "MixDesc":
        return MixDesc(FGD_MIX_IDENTITY, K)

    @staticmethod
    def mean(K: int) -> "MixDesc":
        return MixDesc(FGD_MIX_MEAN, K)

    @staticmethod
    def dense(W) -> "MixDesc":
        W = np.ascontiguousarray(W, dtype=np.float32)
        return MixDesc(FGD_MIX_DENSE, W.shape[0], W=W)

    @staticmethod
    def sparse(nbr, w, w_self, edge_mask=None, renorm: int = FGD_RENORM_NONE) -> "MixDesc":
        nbr = np.ascontiguousarray(nbr, dtype=np.int32)
        K = nbr.shape[0]
        D = nbr.shape[1] if nbr.ndim == 2 else 0
        return MixDesc(FGD_MIX_SPARSE, K, D, renorm, nbr, np.asarray(w, dtype=np.float32),
                       np.asarray(w_self, dtype=np.float32),
                       None if edge_mask is None else np.asarray(edge_mask, dtype=np.uint8))

    @staticmethod
    def _topo(fn, K, D, *args) -> "MixDesc":
        nbr = np.full((K, max(D, 1)), -1, dtype=np.int32)
        w = np.zeros((K, max(D, 1)), dtype=np.float32)
        ws = np.zeros(K, dtype=np.float32)
        rc = fn(K, *args, nbr.ctypes.data, w.ctypes.data, ws.ctypes.data)
        if rc < 0:
            raise FgdError(rc, fgd_last_error(None))
        return MixDesc(FGD_MIX_SPARSE, K, rc, FGD_RENORM_NONE, nbr[:, :rc].copy(), w[:, :rc].copy(), ws)

    @staticmethod
    def ring(K: int) -> "MixDesc":
        return MixDesc._topo(_lib.fgd_topo_ring, K, 2)

    @staticmethod
    def onepeer_xor(K: int, rnd: int) -> "MixDesc":
        return MixDesc._topo(_lib.fgd_topo_onepeer_xor, K, 1, rnd)

    @staticmethod
    def hypercube(K: int) -> "MixDesc":
        return MixDesc._topo(_lib.fgd_topo_hypercube, K, max(1, K.bit_length() - 1))

    @staticmethod
    def random_matching(K: int, seed: int, rnd: int, mix_id: int) -> "MixDesc":
        return MixDesc._topo(_lib.fgd_topo_random_matching, K, 1, seed, rnd, mix_id)

    def with_failures(self, seed: int, rnd: int, mix_id: int, p_fail: float,
                      renorm: int = FGD_RENORM_METROPOLIS) -> "MixDesc":
        """Copy of a sparse descriptor with this round's Bernoulli edge mask attached."""
        mask = fgd_edge_mask(seed, rnd, mix_id, p_fail, self.nbr)
        return MixDesc(FGD_MIX_SPARSE, self.K, self.D, renorm, self.nbr, self.w, self.w_self, mask)


# ------------------------------------------------------------------------ host helpers
def fgd_last_error(ctx) -> str:
    h = ctx._h if isinstance(ctx, Context) else None
    return (_lib.fgd_last_error(h) or b"").decode()


def fgd_hash64(seed: int, rnd: int, tag: int, a: int, b: int) -> int:
    return int(_lib.fgd_hash64(seed, rnd, tag, a, b))


def fgd_edge_mask(seed: int, rnd: int, mix_id: int, p_fail: float, nbr) -> np.ndarray:
    nbr = np.ascontiguousarray(nbr, dtype=np.int32)
    K, D = nbr.shape
    mask = np.zeros((K, D), dtype=np.uint8)
    rc = _lib.fgd_edge_mask(seed, rnd, mix_id, float(p_fail), K, D, nbr.ctypes.data, mask.ctypes.data)
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))
    return mask


def fgd_effective_weights(desc: MixDesc):
    w_eff = np.zeros((desc.K, max(desc.D, 1)), dtype=np.float64)
    ws_eff = np.zeros(desc.K, dtype=np.float64)
    packed = np.zeros(desc.K * max(desc.D, 1), dtype=np.float64)
    rc = _lib.fgd_effective_weights(ctypes.byref(desc.c()), packed.ctypes.data, ws_eff.ctypes.data)
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))
    w_eff = packed[:desc.K * desc.D].reshape(desc.K, desc.D)
    return w_eff, ws_eff


def fgd_dense_matrix(desc: MixDesc) -> np.ndarray:
    W = np.zeros((desc.K, desc.K), dtype=np.float64)
    rc = _lib.fgd_dense_matrix(ctypes.byref(desc.c()), W.ctypes.data)
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))
    return W


def fgd_cd_finalize(sumsq):
    s = np.ascontiguousarray(sumsq, dtype=np.float64)
    a, b = ctypes.c_double(), ctypes.c_double()
    rc = _lib.fgd_cd_finalize(s.ctypes.data, s.shape[0], ctypes.byref(a), ctypes.byref(b))
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))
    return a.value, b.value


# ------------------------------------------------------------------------ GPU entry points
def _dev_ptr(t, name: str, dtype_name: str):
    if t is None:
        return None
    if not getattr(t, "is_cuda", False):
        raise TypeError(f"{name} must be a CUDA tensor")
    if str(t.dtype) != dtype_name:
        raise TypeError(f"{name} must be {dtype_name}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


class Context:
    """Owns one ``fgd_ctx``: fixed K, P, row stride ld and CUDA device."""

    def __init__(self, K: int, P: int, ld: Optional[int] = None, device: int = 0):
        self.K, self.P, self.ld, self.device = int(K), int(P), int(P if ld is None else ld), int(device)
        h = ctypes.c_void_p()
        rc = _lib.fgd_create(ctypes.byref(h), self.device, self.K, self.P, self.ld)
        if rc != 0:
            raise FgdError(rc, fgd_last_error(None))
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            _lib.fgd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != 0:
            raise FgdError(rc, fgd_last_error(self))

    @property
    def launch_count(self) -> int:
        return int(_lib.fgd_launch_count(self._h))


def fgd_set_path(ctx: Context, path: int) -> None:
    ctx._check(_lib.fgd_set_path(ctx._h, int(path)))


FGD_DEBUG_SPIN_LIMIT, FGD_DEBUG_SKIP_TILE, FGD_DEBUG_GOSSIP_PATH = 1, 2, 3


def fgd_debug_set(ctx: Context, key: int, value: int) -> None:
    """Test and measurement hooks: bounded device-side waits, fused-gossip kernel choice (see ``include/fgd.h``)."""
    ctx._check(_lib.fgd_debug_set(ctx._h, int(key), int(value)))


def fgd_debug_stream_pattern(ctx: Context, theta_local, theta_prev, momentum, theta_new, stream=None) -> None:
    """The fused step's HBM traffic without its arithmetic (a measurement aid, see ``include/fgd.h``)."""
    ctx._check(_lib.fgd_debug_stream_pattern(ctx._h, _dev_ptr(theta_local, "theta_local", "torch.float32"),
                                             _dev_ptr(theta_prev, "theta_prev", "torch.float32"),
                                             _dev_ptr(momentum, "momentum", "torch.float32"),
                                             _dev_ptr(theta_new, "theta_new", "torch.float32"), _stream(stream)))


def fgd_device_status(ctx: Context, stream=None) -> None:
    """Synchronises the stream; raises FgdError(FGD_ERR_TIMEOUT) if a device-side wait gave up."""
    ctx._check(_lib.fgd_device_status(ctx._h, _stream(stream)))


def fgd_outer_grad(ctx: Context, theta_prev, theta_local, g, stream=None) -> None:
    ctx._check(_lib.fgd_outer_grad(ctx._h, _dev_ptr(theta_prev, "theta_prev", "torch.float32"),
                                   _dev_ptr(theta_local, "theta_local", "torch.float32"),
                                   _dev_ptr(g, "g", "torch.float32"), _stream(stream)))


def fgd_mix(ctx: Context, desc: MixDesc, inp, out, out_is_vector: bool = False, stream=None) -> None:
    ctx._check(_lib.fgd_mix(ctx._h, ctypes.byref(desc.c()), _dev_ptr(inp, "in", "torch.float32"),
                            _dev_ptr(out, "out", "torch.float32"), int(bool(out_is_vector)), _stream(stream)))


def fgd_outer_step(ctx: Context, mix2: MixDesc, mix1_fused: Optional[MixDesc], x, x_is_vector: bool,
                   theta_local, theta_prev, momentum, theta_new, lr: float = 0.7, mu: float = 0.9,
                   cd_sumsq=None, stream=None) -> None:
    ctx._check(_lib.fgd_outer_step(
        ctx._h, ctypes.byref(mix2.c()), None if mix1_fused is None else ctypes.byref(mix1_fused.c()),
        _dev_ptr(x, "x", "torch.float32"), int(bool(x_is_vector)),
        _dev_ptr(theta_local, "theta_local", "torch.float32"),
        _dev_ptr(theta_prev, "theta_prev", "torch.float32"),
        _dev_ptr(momentum, "momentum", "torch.float32"),
        _dev_ptr(theta_new, "theta_new", "torch.float32"), float(lr), float(mu),
        _dev_ptr(cd_sumsq, "cd_sumsq", "torch.float64"), _stream(stream)))


class _CStepOptions(ctypes.Structure):
    _fields_ = [("mix2_ranges", ctypes.c_void_p), ("n_ranges", ctypes.c_int32), ("average_momentum", ctypes.c_int32),
                ("x_next", ctypes.c_void_p)]


def fgd_outer_step_ex(ctx: Context, mix2: MixDesc, mix1_fused: Optional[MixDesc], x, x_is_vector: bool,
                      theta_local, theta_prev, momentum, theta_new, lr: float = 0.7, mu: float = 0.9,
                      cd_sumsq=None, mix2_ranges=None, average_momentum: bool = False, x_next=None,
                      stream=None) -> None:
    """fgd_outer_step with the paper's two variants: Mix2 only inside the given (lo, hi) column
    ranges (the "-subset" configurations) and/or the momentum averaged first (GlobalM1S); with
    ``x_next`` ([P]) the kernel also writes the column mean of theta_new, i.e. next round's
    global-average Mix1 result."""
    ranges = None
    if mix2_ranges is not None:
        ranges = np.ascontiguousarray(np.asarray(mix2_ranges, dtype=np.int64).reshape(-1, 2))
    opts = _CStepOptions(None if ranges is None else ranges.ctypes.data, 0 if ranges is None else ranges.shape[0],
                         int(bool(average_momentum)), _dev_ptr(x_next, "x_next", "torch.float32"))
    ctx._check(_lib.fgd_outer_step_ex(
        ctx._h, ctypes.byref(mix2.c()), None if mix1_fused is None else ctypes.byref(mix1_fused.c()),
        _dev_ptr(x, "x", "torch.float32"), int(bool(x_is_vector)),
        _dev_ptr(theta_local, "theta_local", "torch.float32"),
        _dev_ptr(theta_prev, "theta_prev", "torch.float32"),
        _dev_ptr(momentum, "momentum", "torch.float32"),
        _dev_ptr(theta_new, "theta_new", "torch.float32"), float(lr), float(mu),
        _dev_ptr(cd_sumsq, "cd_sumsq", "torch.float64"), ctypes.byref(opts), _stream(stream)))


def fgd_outer_step_from_host(ctx: Context, mix2: MixDesc, mix1_fused: Optional[MixDesc], x, x_is_vector: bool,
                             theta_local_host, theta_local_dev, theta_prev, momentum, theta_new,
                             lr: float = 0.7, mu: float = 0.9, want_cd: bool = True, n_chunks: int = 8,
                             stream=None) -> Optional[np.ndarray]:
    """The outer step with theta_local arriving from HOST memory (a CPU tensor [K, ld], pinned for
    full copy bandwidth): copied chunk by chunk into ``theta_local_dev`` while the previous chunk's
    step runs.  With ``want_cd`` the call returns the consensus sums (float64 [K]) after the round
    has completed; without it returns None and is asynchronous."""
    if getattr(theta_local_host, "is_cuda", True) or str(theta_local_host.dtype) != "torch.float32":
        raise TypeError("theta_local_host must be a float32 CPU tensor")
    if theta_local_host.stride(-1) != 1 or (theta_local_host.dim() == 2 and theta_local_host.shape[0] > 1
                                             and theta_local_host.stride(0) != ctx.ld):
        raise ValueError("theta_local_host must be a [K, ld] matrix with the context's row stride")
    cd = np.empty(ctx.K, dtype=np.float64) if want_cd else None
    ctx._check(_lib.fgd_outer_step_from_host(
        ctx._h, ctypes.byref(mix2.c()), None if mix1_fused is None else ctypes.byref(mix1_fused.c()),
        _dev_ptr(x, "x", "torch.float32"), int(bool(x_is_vector)), theta_local_host.data_ptr(),
        _dev_ptr(theta_local_dev, "theta_local_dev", "torch.float32"),
        _dev_ptr(theta_prev, "theta_prev", "torch.float32"),
        _dev_ptr(momentum, "momentum", "torch.float32"),
        _dev_ptr(theta_new, "theta_new", "torch.float32"), float(lr), float(mu),
        None if cd is None else cd.ctypes.data, int(n_chunks), _stream(stream)))
    return cd


def fgd_consensus_distance(ctx: Context, theta, cd_sumsq, stream=None) -> None:
    ctx._check(_lib.fgd_consensus_distance(ctx._h, _dev_ptr(theta, "theta", "torch.float32"),
                                           _dev_ptr(cd_sumsq, "cd_sumsq", "torch.float64"), _stream(stream)))


def fgd_consensus_distance_noalloc(device: int, K: int, P: int, ld: int, theta, cd_sumsq, stream=None) -> None:
    """Consensus sums without a context and without any GPU allocation (for callers that may not
    allocate); partial sums go through a fixed array inside the library, shared by all calls, so
    calls on one GPU must not overlap.  See ``include/fgd.h``."""
    rc = _lib.fgd_consensus_distance_noalloc(int(device), int(K), int(P), int(ld),
                                             _dev_ptr(theta, "theta", "torch.float32"),
                                             _dev_ptr(cd_sumsq, "cd_sumsq", "torch.float64"), _stream(stream))
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))


def fgd_js_distance(worker_logits, avg_logits, top_idx, d_js, cd_worker, top_k: int = 100, device: int = 0,
                    stream=None) -> None:
    """JS functional disagreement of [K, U, V] worker logits against [U, V] averaged-model logits
    on the averaged model's top_k tokens; fills top_idx [U, top_k], d_js [K, U], cd_worker [K]."""
    K, U, V = worker_logits.shape
    rc = _lib.fgd_js_distance(int(device), int(K), int(U), int(V), int(top_k),
                              _dev_ptr(worker_logits, "worker_logits", "torch.float32"),
                              _dev_ptr(avg_logits, "avg_logits", "torch.float32"),
                              _dev_ptr(top_idx, "top_idx", "torch.int32"), _dev_ptr(d_js, "d_js", "torch.float64"),
                              _dev_ptr(cd_worker, "cd_worker", "torch.float64"), _stream(stream))
    if rc != 0:
        raise FgdError(rc, fgd_last_error(None))
