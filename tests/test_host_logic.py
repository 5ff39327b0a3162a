"""CPU tests of the library's host side: exported symbols, topology builders, edge masks and
renormalisation -- compared bit-exactly (indices, masks, hashes) or to 1e-7 (weights) with the
oracle's independent Python implementations."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2606_22768_b200 as fgd
from oracle import topology as T

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "fgd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(fgd_[a-z0-9_]+)\s*\(", header))
    assert {"fgd_outer_grad", "fgd_mix", "fgd_outer_step", "fgd_consensus_distance"} <= declared
    lib = ctypes.CDLL(fgd.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in fgd.h but not exported"
    assert declared == set(fgd.EXPORTED_SYMBOLS), "binding and header disagree"


def test_hash_matches_oracle():
    rng = np.random.default_rng(0)
    for _ in range(200):
        a = [int(x) for x in rng.integers(0, 2 ** 63, 5)]
        assert fgd.fgd_hash64(*a) == T.h64(*a)
    assert fgd.fgd_hash64(2 ** 64 - 1, 0, 1, 2, 3) == T.h64(2 ** 64 - 1, 0, 1, 2, 3)


def _same_topology(desc, ref):
    nbr, w, ws = ref
    assert desc.nbr.tolist() == [list(r[:desc.D]) for r in nbr]
    np.testing.assert_array_equal(desc.w, np.array([r[:desc.D] for r in w], dtype=np.float32))
    np.testing.assert_array_equal(desc.w_self, np.array(ws, dtype=np.float32))


@pytest.mark.parametrize("K", [1, 2, 3, 4, 7, 16, 64])
def test_ring_matches_oracle(K):
    d = fgd.MixDesc.ring(K)
    assert d.D == 2
    _same_topology(d, T.ring(K))


@pytest.mark.parametrize("K", [1, 2, 8, 16, 64])
def test_xor_and_hypercube_match_oracle(K):
    for rnd in range(7):
        _same_topology(fgd.MixDesc.onepeer_xor(K, rnd), T.onepeer_xor(K, rnd))
    _same_topology(fgd.MixDesc.hypercube(K), T.hypercube(K))


def test_non_power_of_two_rejected():
    with pytest.raises(fgd.FgdError) as e:
        fgd.MixDesc.onepeer_xor(6, 0)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError):
        fgd.MixDesc.hypercube(12)
    with pytest.raises(fgd.FgdError):
        fgd.MixDesc.ring(65)


@pytest.mark.parametrize("K", [2, 5, 8, 16, 33])
def test_random_matching_matches_oracle(K):
    for seed in (0, 9):
        for rnd in range(10):
            for mix_id in (1, 2):
                _same_topology(fgd.MixDesc.random_matching(K, seed, rnd, mix_id),
                               T.random_matching(K, seed, rnd, mix_id))


@pytest.mark.parametrize("p_fail", [0.0, 0.05, 0.1, 0.5, 1.0])
def test_edge_mask_bit_exact(p_fail):
    for K, make in ((16, T.hypercube), (16, T.ring), (5, T.ring)):
        nbr, w, ws = make(K)
        for rnd in range(20):
            for mix_id in (1, 2):
                got = fgd.fgd_edge_mask(3, rnd, mix_id, p_fail, np.array(nbr, dtype=np.int32))
                assert got.tolist() == T.edge_mask(3, rnd, mix_id, p_fail, nbr)


@pytest.mark.parametrize("renorm", [fgd.FGD_RENORM_NONE, fgd.FGD_RENORM_SELF_ABSORB, fgd.FGD_RENORM_METROPOLIS])
def test_effective_weights_match_oracle(renorm):
    for K, make in ((16, T.hypercube), (8, T.ring), (2, T.ring)):
        nbr, w, ws = make(K)
        for rnd in range(10):
            mask = T.edge_mask(11, rnd, 2, 0.3, nbr)
            desc = fgd.MixDesc.sparse(nbr, w, ws, mask, renorm)
            w_eff, ws_eff = fgd.fgd_effective_weights(desc)
            w32 = np.array(w, dtype=np.float32).astype(np.float64).tolist()
            ws32 = np.array(ws, dtype=np.float32).astype(np.float64).tolist()
            ref_w, ref_ws = T.effective_weights(nbr, w32, ws32, mask, renorm)
            np.testing.assert_allclose(w_eff, np.array(ref_w), rtol=0, atol=1e-7)
            np.testing.assert_allclose(ws_eff, np.array(ref_ws), rtol=0, atol=1e-7)
            W = fgd.fgd_dense_matrix(desc)
            np.testing.assert_allclose(W, np.array(T.dense_from_sparse(nbr, ref_w, ref_ws)), rtol=0, atol=1e-7)
            if renorm != fgd.FGD_RENORM_NONE:
                assert np.array_equal(W, W.T)
                np.testing.assert_allclose(W.sum(1), 1.0, rtol=0, atol=2e-7)


def test_dense_matrix_of_each_kind():
    np.testing.assert_array_equal(fgd.fgd_dense_matrix(fgd.MixDesc.identity(5)), np.eye(5))
    np.testing.assert_array_equal(fgd.fgd_dense_matrix(fgd.MixDesc.mean(4)), np.full((4, 4), 0.25))
    W = np.arange(9, dtype=np.float32).reshape(3, 3)
    np.testing.assert_array_equal(fgd.fgd_dense_matrix(fgd.MixDesc.dense(W)), W.astype(np.float64))


def test_descriptor_validation():
    nbr, w, ws = T.ring(4)
    bad = [row[:] for row in nbr]
    bad[0][0] = 0                                    # self loop
    with pytest.raises(fgd.FgdError, match="self loop"):
        fgd.fgd_dense_matrix(fgd.MixDesc.sparse(bad, w, ws))
    bad = [row[:] for row in nbr]
    bad[0][0] = 2                                    # 0 -> 2 without 2 -> 0
    with pytest.raises(fgd.FgdError, match="reverse"):
        fgd.fgd_dense_matrix(fgd.MixDesc.sparse(bad, w, ws))
    bad = [row[:] for row in nbr]
    bad[1][0] = 9
    with pytest.raises(fgd.FgdError, match="out of range"):
        fgd.fgd_dense_matrix(fgd.MixDesc.sparse(bad, w, ws))
    mask = [[1, 1] for _ in range(4)]
    mask[0][1] = 0                                   # edge {0,1} dropped on one side only
    with pytest.raises(fgd.FgdError, match="symmetric"):
        fgd.fgd_dense_matrix(fgd.MixDesc.sparse(nbr, w, ws, mask))
    dup = [[1, 1], [0, 0], [3, 3], [2, 2]]
    with pytest.raises(fgd.FgdError, match="twice"):
        fgd.fgd_dense_matrix(fgd.MixDesc.sparse(dup, w, ws))


def test_cd_finalize():
    n, q = fgd.fgd_cd_finalize([4.0, 9.0, 0.0, 1.0])
    assert n == 1.5 and q == 3.5
    assert fgd.fgd_cd_finalize([1.0])[0] == 1.0


def test_gpu_entry_points_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(fgd.FgdError) as e:
        fgd.Context(4, 128)
    assert e.value.status == fgd.FGD_ERR_CUDA


def _random_graph(rng, K, max_deg):
    """Random undirected graph as padded neighbour lists (-1 = empty slot), Metropolis base weights."""
    adj = [[] for _ in range(K)]
    pairs = [(a, b) for a in range(K) for b in range(a + 1, K)]
    rng.shuffle(pairs)
    for a, b in pairs:
        if len(adj[a]) < max_deg and len(adj[b]) < max_deg and rng.random() < 0.5:
            adj[a].append(b)
            adj[b].append(a)
    D = max(1, max(len(r) for r in adj))
    nbr = [r + [-1] * (D - len(r)) for r in adj]
    deg = [len(r) for r in adj]
    w = [[(1.0 / (1 + max(deg[m], deg[n])) if n >= 0 else 0.0) for n in nbr[m]] for m in range(K)]
    ws = [1.0 - sum(w[m]) for m in range(K)]
    return nbr, w, ws


@pytest.mark.parametrize("renorm", [fgd.FGD_RENORM_NONE, fgd.FGD_RENORM_SELF_ABSORB, fgd.FGD_RENORM_METROPOLIS])
def test_masks_and_renormalisation_on_random_graphs(renorm):
    """Irregular degrees, empty slots, every drop rate: the two implementations agree (masks bit for
    bit, weights to 1e-7) and the invariants of the reading hold -- symmetric, non-negative, and
    doubly stochastic under both renormalisation rules."""
    rng = np.random.default_rng(2024)
    for trial in range(40):
        K = int(rng.integers(3, 65))
        nbr, w, ws = _random_graph(rng, K, int(rng.integers(1, fgd.FGD_MAX_D + 1)))
        p_fail = float(rng.choice([0.0, 0.05, 0.3, 0.7, 1.0]))
        nbr_np = np.array(nbr, dtype=np.int32)
        mask = T.edge_mask(trial, 3 * trial, 1 + trial % 2, p_fail, nbr)
        assert fgd.fgd_edge_mask(trial, 3 * trial, 1 + trial % 2, p_fail, nbr_np).tolist() == mask
        desc = fgd.MixDesc.sparse(nbr, w, ws, mask, renorm)
        w_eff, ws_eff = fgd.fgd_effective_weights(desc)
        w32 = np.array(w, dtype=np.float32).astype(np.float64).tolist()
        ws32 = np.array(ws, dtype=np.float32).astype(np.float64).tolist()
        ref_w, ref_ws = T.effective_weights(nbr, w32, ws32, mask, renorm)
        np.testing.assert_allclose(w_eff, np.array(ref_w), rtol=0, atol=1e-7)
        np.testing.assert_allclose(ws_eff, np.array(ref_ws), rtol=0, atol=1e-7)
        W = fgd.fgd_dense_matrix(desc)
        assert np.array_equal(W, W.T) and (W >= -1e-7).all()
        if renorm != fgd.FGD_RENORM_NONE:
            np.testing.assert_allclose(W.sum(0), 1.0, rtol=0, atol=4e-7)
            np.testing.assert_allclose(W.sum(1), 1.0, rtol=0, atol=4e-7)
        if p_fail == 1.0 and renorm != fgd.FGD_RENORM_NONE:
            np.testing.assert_allclose(W, np.eye(K), rtol=0, atol=4e-7)     # every exchange failed: nobody mixes
