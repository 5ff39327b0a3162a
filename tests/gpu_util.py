"""Shared helpers of the GPU parity tests: build the same mix on both sides (library builders
for the CUDA path, oracle builders for the reference), run rounds on both, compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen
from oracle import topology as T
from paper_2606_22768_b200.round import OuterRound

RTOL, ATOL = 1e-5, 1e-7  # fp32 parameters: max relative error 1e-5, absolute 1e-7 near zero
CD_RTOL = 1e-5


def assert_param_close(got, ref, what=""):
    """Element-wise: |got - ref| <= 1e-7 or |got - ref| <= 1e-5 |ref|."""
    got = got.detach().double().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, f"{what}: shape {got.shape} vs {ref.shape}"
    err = np.abs(got - ref)
    bad = ~((err <= ATOL) | (err <= RTOL * np.abs(ref)))
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err, 0)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} elements out of tolerance; worst at {i}: "
                             f"got {got[i]!r} ref {ref[i]!r} err {err[i]:.3e}")


def assert_cd_close(got, ref, P, what=""):
    got = got.detach().cpu().numpy() if isinstance(got, torch.Tensor) else np.asarray(got)
    ref = np.asarray(ref, dtype=np.float64)
    floor = 1e-12 * P  # exact-consensus cases: fp32 means of equal values are off by an ulp
    # theta_new and the column mean are each rounded to fp32 (a few ulps of |theta| <= 0.1, delta <= 8e-9)
    # before the deviation d is squared: s moves by about 2 delta sqrt(s) (random signs), which only
    # matters when there are so few columns that nothing averages out; 4 sigma of that.
    # That term is derived for, and applies to, inputs of at most 64 columns only.
    rounding = 8 * 8e-9 * np.sqrt(np.abs(ref)) if P <= 64 else np.zeros_like(ref)
    err = np.abs(got - ref)
    assert ((err <= CD_RTOL * np.abs(ref)) | (err <= floor) | (err <= rounding)).all(), f"{what}: got {got} ref {ref}"


def make_mix(spec, K, rnd, seed, mix_id):
    """spec -> (MixDesc built with the LIBRARY's helpers, dense float64 W built with the ORACLE's)."""
    kind = spec[0]
    if kind == "identity":
        return fgd.MixDesc.identity(K), oracle.dense_W("identity", K)
    if kind == "mean":
        return fgd.MixDesc.mean(K), oracle.dense_W("mean", K)
    if kind == "dense":
        W32 = np.asarray(spec[1], dtype=np.float32)
        return fgd.MixDesc.dense(W32), oracle.dense_W("dense", K, W=W32.astype(np.float64))
    if kind == "circulant":   # neighbours m +- 1 .. m +- h (D = 2h slots), Metropolis weights 1/(1+2h)
        h = spec[1]
        p_fail = spec[2] if len(spec) > 2 else 0.0
        renorm = spec[3] if len(spec) > 3 else fgd.FGD_RENORM_METROPOLIS
        nbr = [[(m + s * d) % K for d in range(1, h + 1) for s in (-1, 1)] for m in range(K)]
        w = [[1.0 / (1 + 2 * h)] * (2 * h) for _ in range(K)]
        ws = [1.0 / (1 + 2 * h)] * K
        d = fgd.MixDesc.sparse(nbr, w, ws)
        w32 = np.array(w, dtype=np.float32).astype(np.float64).tolist()
        ws32 = np.array(ws, dtype=np.float32).astype(np.float64).tolist()
        mask = None
        if p_fail > 0.0:
            d = d.with_failures(seed, rnd, mix_id, p_fail, renorm)
            mask = T.edge_mask(seed, rnd, mix_id, p_fail, nbr)
            assert d.edge_mask.tolist() == mask
        w_eff, ws_eff = T.effective_weights(nbr, w32, ws32, mask, renorm if mask is not None else T.RENORM_NONE)
        return d, np.array(T.dense_from_sparse(nbr, w_eff, ws_eff), dtype=np.float64)
    if kind == "randgraph":   # seeded irregular graph: degrees 0..max_deg, empty slots, Metropolis base weights
        max_deg = spec[1]
        p_fail = spec[2] if len(spec) > 2 else 0.0
        rng = np.random.default_rng(1000 * K + max_deg)
        adj = [[] for _ in range(K)]
        pairs = [(a, b) for a in range(K) for b in range(a + 1, K)]
        rng.shuffle(pairs)
        for a, b in pairs:
            if len(adj[a]) < max_deg and len(adj[b]) < max_deg and rng.random() < 0.6:
                adj[a].append(b)
                adj[b].append(a)
        D = max(1, max(len(r) for r in adj))
        nbr = [r + [-1] * (D - len(r)) for r in adj]
        deg = [len(r) for r in adj]
        w = [[(1.0 / (1 + max(deg[m], deg[n])) if n >= 0 else 0.0) for n in nbr[m]] for m in range(K)]
        ws = [1.0 - sum(w[m]) for m in range(K)]
        d = fgd.MixDesc.sparse(nbr, w, ws)
        w32 = np.array(w, dtype=np.float32).astype(np.float64).tolist()
        ws32 = np.array(ws, dtype=np.float32).astype(np.float64).tolist()
        mask = None
        if p_fail > 0.0:
            d = d.with_failures(seed, rnd, mix_id, p_fail, fgd.FGD_RENORM_METROPOLIS)
            mask = T.edge_mask(seed, rnd, mix_id, p_fail, nbr)
            assert d.edge_mask.tolist() == mask
        w_eff, ws_eff = T.effective_weights(nbr, w32, ws32, mask, T.RENORM_METROPOLIS if mask is not None else T.RENORM_NONE)
        return d, np.array(T.dense_from_sparse(nbr, w_eff, ws_eff), dtype=np.float64)
    if kind == "isolated":    # a sparse descriptor with no neighbour slots at all (D = 0): W = I
        d = fgd.MixDesc.sparse(np.zeros((K, 0), dtype=np.int32), np.zeros((K, 0), dtype=np.float32), np.ones(K, dtype=np.float32))
        return d, oracle.dense_W("identity", K)
    if kind in ("ring", "xor", "hypercube", "matching"):
        p_fail = spec[1] if len(spec) > 1 else 0.0
        renorm = spec[2] if len(spec) > 2 else fgd.FGD_RENORM_METROPOLIS
        if kind == "ring":
            d, (nbr, w, ws) = fgd.MixDesc.ring(K), T.ring(K)
        elif kind == "xor":
            d, (nbr, w, ws) = fgd.MixDesc.onepeer_xor(K, rnd), T.onepeer_xor(K, rnd)
        elif kind == "hypercube":
            d, (nbr, w, ws) = fgd.MixDesc.hypercube(K), T.hypercube(K)
        else:
            d, (nbr, w, ws) = fgd.MixDesc.random_matching(K, seed, rnd, mix_id), T.random_matching(K, seed, rnd, mix_id)
        # the oracle sees the base weights as the fp32 values the caller hands the library
        w32 = np.array(w, dtype=np.float32).astype(np.float64).tolist()
        ws32 = np.array(ws, dtype=np.float32).astype(np.float64).tolist()
        mask = None
        if p_fail > 0.0:
            d = d.with_failures(seed, rnd, mix_id, p_fail, renorm)
            mask = T.edge_mask(seed, rnd, mix_id, p_fail, nbr)
            assert d.edge_mask.tolist() == mask, "edge masks must agree bit for bit"
        w_eff, ws_eff = T.effective_weights(nbr, w32, ws32, mask, renorm if mask is not None else T.RENORM_NONE)
        return d, np.array(T.dense_from_sparse(nbr, w_eff, ws_eff), dtype=np.float64)
    raise ValueError(spec)


def padded(K, P, ld, fill=np.float32(-777.0)):
    """[K, ld] CUDA tensor filled with a sentinel; returns (full tensor, [K, P] view)."""
    full = torch.full((K, ld), float(fill), dtype=torch.float32, device="cuda")
    return full, full[:, :P]


def upload(a32, ld):
    K, P = a32.shape
    full, view = padded(K, P, ld)
    view.copy_(torch.from_numpy(np.ascontiguousarray(a32)))
    return full, view


def check_padding(full, P, what=""):
    if full.shape[1] > P:
        assert bool((full[:, P:] == -777.0).all()), f"{what}: padding columns were written"


class Scenario:
    """Runs R free-running rounds on the GPU and in the oracle from the same seeded inputs and
    compares theta_new, momentum and the consensus sums after every round."""

    def __init__(self, K, P, mix1, mix2, *, ld=None, seed=0, sigmas=1e-3, worker_std=0.0, mode="factored",
                 in_place=True, lr=0.7, mu=0.9, v0_std=0.0, path=fgd.FGD_PATH_AUTO,
                 mix2_ranges=None, average_momentum=False, chain_mix1=False):
        self.K, self.P, self.ld = K, P, P if ld is None else ld
        self.mix1, self.mix2, self.seed, self.mode, self.in_place = mix1, mix2, seed, mode, in_place
        self.lr, self.mu = lr, mu
        self.mix2_ranges, self.average_momentum = mix2_ranges, average_momentum
        self.chain_mix1 = chain_mix1   # rounds > 0 take Mix1 (mean) from the previous step's x_next
        self.sigmas = np.broadcast_to(np.asarray(sigmas, dtype=np.float32), (K,)).copy()
        th0 = gen.theta0(seed, K, P, 0.02, worker_std)
        v0 = (gen.scaled_normal(seed, gen.TENSOR_MOMENTUM, 0, K, P, v0_std) if v0_std > 0
              else np.zeros((K, P), dtype=np.float32))
        self.o_theta, self.o_v = th0.astype(np.float64), v0.astype(np.float64)
        self.full_prev, self.g_prev = upload(th0, self.ld)
        self.full_v, self.g_v = upload(v0, self.ld)
        self.full_loc, self.g_loc = padded(K, P, self.ld)
        self.full_new, self.g_new = (self.full_prev, self.g_prev) if in_place else padded(K, P, self.ld)
        self.drv = OuterRound(K, P, self.ld)
        fgd.fgd_set_path(self.drv.ctx, path)

    def run(self, R):
        K, P = self.K, self.P
        for r in range(R):
            m1_desc, W1 = make_mix(self.mix1, K, r, self.seed, 1)
            m2_desc, W2 = make_mix(self.mix2, K, r, self.seed, 2)
            # stand-in for the inner steps: same fp32 drift bits on both sides
            drift = gen.scaled_normal(self.seed, gen.TENSOR_DRIFT, r, K, P, self.sigmas)
            fused = self.mode == "fused" or self.mix1[0] == "identity"
            if not fused and not (self.chain_mix1 and r > 0):
                self.drv.launch_mix1(m1_desc, self.full_prev)
            th_prev32 = self.g_prev.cpu().numpy()
            loc32 = th_prev32 + drift
            self.g_loc.copy_(torch.from_numpy(loc32))
            self.drv.step(m2_desc, self.full_loc, self.full_prev, self.full_v, self.full_new, self.lr, self.mu,
                          mix1_fused=m1_desc if fused else None, want_cd=True,
                          mix2_ranges=self.mix2_ranges, average_momentum=self.average_momentum,
                          emit_next_mix1=self.chain_mix1)
            torch.cuda.synchronize()
            # oracle, free running: its own float64 state plus the shared drift
            o_loc = self.o_theta + drift.astype(np.float64)
            if self.mix2_ranges is None and not self.average_momentum:
                self.o_theta, self.o_v = oracle.outer_round(W1, W2, self.o_theta, o_loc, self.o_v, self.lr, self.mu)
            else:
                self.o_theta, self.o_v = oracle.outer_round_ex(W1, W2, self.o_theta, o_loc, self.o_v, self.lr, self.mu,
                                                               self.mix2_ranges, self.average_momentum)
            assert_param_close(self.g_new, self.o_theta, f"theta_new round {r}")
            assert_param_close(self.g_v, self.o_v, f"momentum round {r}")
            assert_cd_close(self.drv.cd_sumsq, oracle.consensus_sumsq(self.o_theta), P, f"cd_sumsq round {r}")
            for full, name in ((self.full_new, "theta_new"), (self.full_v, "momentum"), (self.full_loc, "theta_local")):
                check_padding(full, P, name)
            if not self.in_place:
                self.g_prev.copy_(self.g_new)
        fgd.fgd_device_status(self.drv.ctx)
        return self
