"""Pins of the float64 oracle against what the paper and the mathematics fix (CPU only).

Each test ties the oracle to something other than itself: a hand-worked fixture, a
library routine (numpy matmul / eigvalsh, torch.optim.SGD), a closed form, an invariant,
or brute force on tiny inputs.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import topology as T
from fgd_inputs import gen
from tests.conftest import read_golden

GAMMA, MU = 0.7, 0.9


def _vals(d, key):
    return np.array([float(Fraction(s)) for s in d[key]], dtype=np.float64)


def _rand(K, P, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal((K, P)) * scale


def _ring_W(K):
    nbr, w, ws = T.ring(K)
    return np.array(T.dense_from_sparse(nbr, w, ws))


def _hyper_W(K):
    nbr, w, ws = T.hypercube(K)
    return np.array(T.dense_from_sparse(nbr, w, ws))


# ------------------------------------------------------------------ worked example
def test_worked_round_fixture():
    """Two consecutive rounds worked by hand (K=4, P=1, Mix1 mean, Mix2 ring 1/3)."""
    d = read_golden("worked_round_ring4.txt")
    K = int(d["K"][0])
    W1 = oracle.dense_W("mean", K)
    W2 = _ring_W(K)
    tp = _vals(d, "r0.theta_prev").reshape(K, 1)
    v = _vals(d, "r0.v").reshape(K, 1)
    for r in ("r0", "r1"):
        tl = _vals(d, f"{r}.theta_local").reshape(K, 1)
        tn, v, x, gh = oracle.outer_round(W1, W2, tp, tl, v, GAMMA, MU, want_intermediates=True)
        np.testing.assert_allclose(gh[:, 0], _vals(d, f"{r}.ghat"), rtol=0, atol=1e-15)
        np.testing.assert_allclose(x[:, 0], _vals(d, f"{r}.x"), rtol=0, atol=1e-15)
        np.testing.assert_allclose(v[:, 0], _vals(d, f"{r}.v_new"), rtol=0, atol=1e-15)
        np.testing.assert_allclose(tn[:, 0], _vals(d, f"{r}.theta_new"), rtol=0, atol=2e-15)
        s = oracle.consensus_sumsq(tn)
        np.testing.assert_allclose(s, _vals(d, f"{r}.sumsq"), rtol=1e-12)
        cd_norm, cd_sq = oracle.cd_finalize(s)
        assert cd_norm == pytest.approx(float(d[f"{r}.cd_norm"][0]), rel=1e-12)
        assert cd_sq == pytest.approx(float(d[f"{r}.cd_sq"][0]), rel=1e-12)
        tp = tn


def test_round_brute_force_rationals():
    """K=3, P=5 with NON-symmetric W1, W2 (row convention), exact rational arithmetic.

    A transposed operand, a swapped W1/W2, a sign slip or a dropped mu term all fail here.
    """
    K, P = 3, 5
    W1 = [[Fraction(1, 2), Fraction(1, 2), 0], [0, Fraction(1, 4), Fraction(3, 4)], [Fraction(1, 3), Fraction(1, 3), Fraction(1, 3)]]
    W2 = [[Fraction(1, 5), Fraction(4, 5), 0], [Fraction(1, 2), 0, Fraction(1, 2)], [0, Fraction(1, 8), Fraction(7, 8)]]
    rng = np.random.default_rng(5)
    as_frac = lambda a: [[Fraction(int(x), 64) for x in row] for row in a]
    tp = as_frac(rng.integers(-200, 200, (K, P)))
    tl = as_frac(rng.integers(-200, 200, (K, P)))
    v = as_frac(rng.integers(-50, 50, (K, P)))
    ga, mu = Fraction(7, 10), Fraction(9, 10)
    exp_t = [[None] * P for _ in range(K)]
    exp_v = [[None] * P for _ in range(K)]
    for p in range(P):
        g = [tp[m][p] - tl[m][p] for m in range(K)]
        for m in range(K):
            x = sum(W1[m][n] * tp[n][p] for n in range(K))
            gh = sum(W2[m][n] * g[n] for n in range(K))
            vn = mu * v[m][p] + gh
            exp_v[m][p] = vn
            exp_t[m][p] = x - ga * (gh + mu * vn)
    f = lambda a: np.array([[float(x) for x in row] for row in a])
    tn, vn = oracle.outer_round(f(W1), f(W2), f(tp), f(tl), f(v), 0.7, 0.9)
    np.testing.assert_allclose(tn, f(exp_t), rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(vn, f(exp_v), rtol=1e-14, atol=1e-14)
    # the transposed matrices give a different answer, so the test can see a transposition
    tn_T, _ = oracle.outer_round(f(W1).T, f(W2).T, f(tp), f(tl), f(v), 0.7, 0.9)
    assert np.abs(tn_T - tn).max() > 1e-3


# ------------------------------------------------------------------ library-routine pins
def _torch_nesterov_steps(x0, grads, lr=GAMMA, mu=MU):
    """torch.optim.SGD(nesterov=True) in float64 on CPU, one step per gradient."""
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, nesterov=True)
    outs = []
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        outs.append(p.detach().numpy().copy())
    return outs


def test_identity_mixes_are_independent_torch_sgd():
    """W1 = W2 = I: every worker is its own SGD-Nesterov run (App. B says the update is
    PyTorch's), over three rounds so the momentum buffer matters."""
    K, P, R = 3, 40, 3
    I = oracle.dense_W("identity", K)
    tp = _rand(K, P, 1, 0.02)
    v = np.zeros((K, P))
    drifts = [_rand(K, P, 10 + r, 1e-3) for r in range(R)]
    # gradient of round r depends on theta_prev of round r: replay torch per worker
    ours = []
    cur, curv = tp.copy(), v.copy()
    for r in range(R):
        tl = cur + drifts[r]
        cur, curv = oracle.outer_round(I, I, cur, tl, curv, GAMMA, MU)
        ours.append(cur.copy())
    for m in range(K):
        # identity mixes: g_r = theta_prev_r - theta_local_r = -drift_r, independent of the state
        outs = _torch_nesterov_steps(tp[m], [-drifts[r][m] for r in range(R)])
        for r in range(R):
            np.testing.assert_allclose(ours[r][m], outs[r], rtol=1e-13, atol=1e-16)


def test_global_mixes_reduce_to_diloco():
    """W1 = W2 = (1/K) 1 1^T with identical momentum rows: every worker ends on DiLoCo's
    x_{r+1} = OuterOpt(x_r, -mean_m Delta_m), and the consensus distance is zero."""
    K, P = 8, 64
    J = oracle.dense_W("mean", K)
    base = _rand(1, P, 2, 0.02)
    tp = np.repeat(base, K, axis=0)
    v0 = np.repeat(_rand(1, P, 3, 1e-3), K, axis=0)
    tl = tp + _rand(K, P, 4, 1e-3)
    tn, vn = oracle.outer_round(J, J, tp, tl, v0, GAMMA, MU)
    delta_bar = (tl - tp).mean(axis=0)
    p = torch.nn.Parameter(torch.tensor(base[0], dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=GAMMA, momentum=MU, nesterov=True)
    opt.state[p]["momentum_buffer"] = torch.tensor(v0[0], dtype=torch.float64)
    p.grad = torch.tensor(-delta_bar, dtype=torch.float64)
    opt.step()
    for m in range(K):
        np.testing.assert_allclose(tn[m], p.detach().numpy(), rtol=1e-12, atol=1e-16)
    s = oracle.consensus_sumsq(tn)
    assert s.max() < 1e-28


def test_mix_matches_numpy_matmul():
    """Mix_W(v) with rows as workers is the matrix product W @ V (row convention)."""
    K, P = 7, 33
    W = np.random.default_rng(0).random((K, K))
    V = _rand(K, P, 1)
    np.testing.assert_allclose(oracle.mix(W, V), W @ V, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(oracle.mix(oracle.dense_W("mean", K), V),
                               np.repeat(V.mean(axis=0, keepdims=True), K, 0), rtol=1e-13, atol=1e-15)
    assert np.array_equal(oracle.mix(oracle.dense_W("identity", K), V), V)


def test_outer_grad_sign_and_definition():
    tp, tl = _rand(4, 9, 1), _rand(4, 9, 2)
    assert np.array_equal(oracle.outer_grad(tp, tl), tp - tl)


def test_gamma1_mu0_is_factored_formulation():
    """gamma=1, mu=0: z' = Mix1(z) + Mix2(Delta) with Delta = y_H - y_0 (Sec. 4.1; App. E)."""
    K, P = 6, 21
    W1, W2 = _ring_W(K), gen.sinkhorn_W(3, K).astype(np.float64)
    tp, tl = _rand(K, P, 1), _rand(K, P, 2)
    tn, vn = oracle.outer_round(W1, W2, tp, tl, _rand(K, P, 3), 1.0, 0.0)
    np.testing.assert_allclose(tn, W1 @ tp + W2 @ (tl - tp), rtol=1e-13, atol=1e-14)


def test_nesterov_closed_form():
    """x - gamma (g + mu (mu v + g)) == x - gamma ((1 + mu) g + mu^2 v) (App. B, third line)."""
    x, g, v = _rand(3, 11, 1), _rand(3, 11, 2), _rand(3, 11, 3)
    tn, vn = oracle.nesterov(x, g, v, GAMMA, MU)
    np.testing.assert_allclose(tn, x - GAMMA * ((1 + MU) * g + MU * MU * v), rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(vn, MU * v + g, rtol=1e-15)


# ------------------------------------------------------------------ invariants
@pytest.mark.parametrize("make", [lambda: _ring_W(16), lambda: _hyper_W(16),
                                  lambda: gen.sinkhorn_W(0, 64).astype(np.float64)])
def test_doubly_stochastic_preserves_mean(make):
    W = make()
    K = W.shape[0]
    V = _rand(K, 50, 7)
    np.testing.assert_allclose(oracle.mix(W, V).mean(axis=0), V.mean(axis=0), rtol=0, atol=K * 1e-7)


def test_whole_round_mean_identity():
    """For doubly-stochastic W1, W2 the worker mean obeys the plain Nesterov recursion:
    mean theta_new = mean theta_prev - gamma ((1+mu) mean g + mu^2 mean v) (Sec. 4.2 + App. B)."""
    K, P = 16, 30
    W1, W2 = _hyper_W(K), _ring_W(K)
    tp, tl, v = _rand(K, P, 1, 0.02), _rand(K, P, 2, 0.02), _rand(K, P, 3, 1e-3)
    tn, _ = oracle.outer_round(W1, W2, tp, tl, v, GAMMA, MU)
    expect = tp.mean(0) - GAMMA * ((1 + MU) * (tp - tl).mean(0) + MU * MU * v.mean(0))
    np.testing.assert_allclose(tn.mean(0), expect, rtol=0, atol=1e-15)


def test_contraction_factor_constants():
    """||X W - Xbar||_F^2 <= lambda_2(W)^2 ||X - Xbar||_F^2, with the closed-form constants."""
    d = read_golden("spectral_constants.txt")
    for name, W in (("ring.K4", _ring_W(4)), ("ring.K16", _ring_W(16)), ("hypercube.K16", _hyper_W(16))):
        K = W.shape[0]
        ev = np.sort(np.abs(np.linalg.eigvalsh(W)))
        rho = ev[-2] ** 2
        assert rho == pytest.approx(float(d[name + ".rho"][0]), rel=1e-9)
        assert (W * W).sum() - 1 == pytest.approx(float(d[name + ".frob2_minus_1"][0]), rel=1e-12)
        X = _rand(K, 200, 11)
        Xbar = np.repeat(X.mean(0, keepdims=True), K, 0)
        mixed = oracle.mix(W, X)
        ratio = ((mixed - Xbar) ** 2).sum() / ((X - Xbar) ** 2).sum()
        assert ratio <= rho * (1 + 1e-12)
        # the bound is attained on the second eigenvector
        w, U = np.linalg.eigh(W)
        u2 = U[:, np.argsort(np.abs(w))[-2]].reshape(K, 1)
        assert ((oracle.mix(W, u2) ** 2).sum() / (u2 ** 2).sum()) == pytest.approx(rho, rel=1e-9)


def _all_perfect_matchings(items):
    if not items:
        yield []
        return
    a = items[0]
    for i in range(1, len(items)):
        rest = items[1:i] + items[i + 1:]
        for m in _all_perfect_matchings(rest):
            yield [(a, items[i])] + m


@pytest.mark.parametrize("M", [4, 6, 8])
def test_random_matching_expected_contraction(M):
    """Averaged over ALL perfect matchings the contraction is exactly (M-2)/(2(M-1)) (Sec. 3)."""
    d = read_golden("spectral_constants.txt")
    X = _rand(M, 17, 3)
    Xbar = np.repeat(X.mean(0, keepdims=True), M, 0)
    den = ((X - Xbar) ** 2).sum()
    ratios = []
    for match in _all_perfect_matchings(list(range(M))):
        nbr = [[-1] for _ in range(M)]
        w = [[0.0] for _ in range(M)]
        ws = [1.0] * M
        for a, b in match:
            nbr[a][0], nbr[b][0] = b, a
            w[a][0] = w[b][0] = 0.5
            ws[a] = ws[b] = 0.5
        W = np.array(T.dense_from_sparse(nbr, w, ws))
        ratios.append(((oracle.mix(W, X) - Xbar) ** 2).sum() / den)
    assert len(ratios) == math.prod(range(M - 1, 0, -2))
    assert np.mean(ratios) == pytest.approx((M - 2) / (2 * (M - 1)), rel=1e-12)
    assert np.mean(ratios) == pytest.approx(float(d[f"matching.M{M}.rho_bar"][0]), rel=1e-12)


def test_random_matching_builder_is_a_matching_and_roughly_uniform():
    for K in (2, 5, 8, 9):
        counts = {}
        for rnd in range(300 if K == 5 else 20):
            nbr, w, ws = T.random_matching(K, 7, rnd, 2)
            partner = [row[0] for row in nbr]
            unmatched = [m for m in range(K) if partner[m] < 0]
            assert len(unmatched) == K % 2
            for m in range(K):
                if partner[m] >= 0:
                    assert partner[partner[m]] == m and partner[m] != m
                    assert w[m][0] == 0.5 and ws[m] == 0.5
                else:
                    assert ws[m] == 1.0
            W = np.array(T.dense_from_sparse(nbr, w, ws))
            assert np.array_equal(W, W.T) and np.allclose(W.sum(1), 1)
            counts[tuple(partner)] = counts.get(tuple(partner), 0) + 1
        if K == 5:  # 15 matchings of 5 workers (one idle); each should show up
            assert len(counts) == 15 and max(counts.values()) < 3 * 300 / 15


@pytest.mark.parametrize("K", [2, 4, 8, 16, 64])
def test_onepeer_xor_product_is_global_average(K):
    """log2(K) consecutive one-peer rounds multiply to (1/K) 1 1^T exactly (dyadic weights)."""
    prod = np.eye(K)
    for r in range(K.bit_length() - 1):
        nbr, w, ws = T.onepeer_xor(K, r)
        prod = np.array(T.dense_from_sparse(nbr, w, ws)) @ prod
    assert np.array_equal(prod, np.full((K, K), 1.0 / K))


def test_topology_shapes():
    nbr, w, ws = T.ring(16)
    assert nbr[0] == [15, 1] and nbr[15] == [14, 0] and w[3] == [1 / 3, 1 / 3]
    assert T.ring(2)[0] == [[1, -1], [0, -1]] and T.ring(1)[2] == [1.0]
    nbr, w, ws = T.hypercube(16)
    assert nbr[5] == [4, 7, 1, 13] and ws[0] == pytest.approx(0.2)
    assert T.onepeer_xor(8, 4)[0][3] == [3 ^ 2]  # round 4 -> bit 4 mod 3 = 1
    with pytest.raises(ValueError):
        T.onepeer_xor(6, 0)
    for W in (_ring_W(4), _ring_W(2), _ring_W(16), _hyper_W(8)):
        assert np.array_equal(W, W.T) and np.allclose(W.sum(1), 1.0, atol=1e-15) and (W >= 0).all()


# ------------------------------------------------------------------ edge failures
def test_hash_is_splitmix64():
    """mix64 over the golden-ratio sequence is the splitmix64 generator; its first outputs
    for seed 0 are a widely published test vector."""
    assert T.mix64(T.GOLDEN) == 0xE220A8397B1DCDAF
    assert T.mix64((2 * T.GOLDEN) & T.MASK64) == 0x6E789E6AA1B965F4
    assert T.mix64((3 * T.GOLDEN) & T.MASK64) == 0x06C45D188009454F


def _frac_rows(d, prefix, K):
    return np.array([[float(Fraction(s)) for s in d[f"{prefix}.row{m}"]] for m in range(K)])


def _mask_dropping(nbr, dropped):
    dead = {tuple(sorted(e)) for e in dropped}
    return [[0 if (n < 0 or tuple(sorted((m, n))) in dead) else 1 for n in row] for m, row in enumerate(nbr)]


def test_worked_renormalisation_fixture():
    d = read_golden("worked_renorm.txt")
    nbr, w, ws = T.hypercube(8)
    mask = _mask_dropping(nbr, [(0, 1), (2, 3)])
    for rule, key in ((T.RENORM_METROPOLIS, "A.metropolis"), (T.RENORM_SELF_ABSORB, "A.self_absorb")):
        W = np.array(T.dense_from_sparse(nbr, *T.effective_weights(nbr, w, ws, mask, rule)))
        np.testing.assert_allclose(W, _frac_rows(d, key, 8), rtol=0, atol=1e-15)
    nbr, w, ws = T.ring(4)
    mask = _mask_dropping(nbr, [(0, 1)])
    for rule in (T.RENORM_METROPOLIS, T.RENORM_SELF_ABSORB):
        W = np.array(T.dense_from_sparse(nbr, *T.effective_weights(nbr, w, ws, mask, rule)))
        np.testing.assert_allclose(W, _frac_rows(d, "B", 4), rtol=0, atol=1e-15)


@pytest.mark.parametrize("rule", [T.RENORM_METROPOLIS, T.RENORM_SELF_ABSORB])
def test_masked_matrices_stay_symmetric_doubly_stochastic(rule):
    nbr, w, ws = T.hypercube(16)
    for rnd in range(30):
        mask = T.edge_mask(5, rnd, 2, 0.3, nbr)
        for m in range(16):  # the mask itself is symmetric
            for j, n in enumerate(nbr[m]):
                assert mask[m][j] == mask[n][nbr[n].index(m)]
        w_eff, ws_eff = T.effective_weights(nbr, w, ws, mask, rule)
        W = np.array(T.dense_from_sparse(nbr, w_eff, ws_eff))
        assert np.array_equal(W, W.T) and (W >= 0).all()
        np.testing.assert_allclose(W.sum(1), 1.0, rtol=0, atol=1e-15)
        for m in range(16):
            for j in range(4):
                assert (w_eff[m][j] == 0.0) == (mask[m][j] == 0)


def test_mask_extremes_and_rate():
    nbr, w, ws = T.hypercube(16)
    all_alive = T.edge_mask(1, 0, 1, 0.0, nbr)
    assert all(all(x == 1 for x in row) for row in all_alive)
    for rule in (T.RENORM_NONE, T.RENORM_SELF_ABSORB, T.RENORM_METROPOLIS):
        W = np.array(T.dense_from_sparse(nbr, *T.effective_weights(nbr, w, ws, all_alive, rule)))
        np.testing.assert_allclose(W, _hyper_W(16), rtol=0, atol=1e-15)
    none_alive = T.edge_mask(1, 0, 1, 1.0, nbr)
    assert all(all(x == 0 for x in row) for row in none_alive)
    for rule in (T.RENORM_SELF_ABSORB, T.RENORM_METROPOLIS):
        W = np.array(T.dense_from_sparse(nbr, *T.effective_weights(nbr, w, ws, none_alive, rule)))
        np.testing.assert_allclose(W, np.eye(16), rtol=0, atol=1e-15)
    assert T.drop_threshold(0.1) == 429496729
    # drop rate of p = 0.1 over 32 edges x 400 rounds, within 4 binomial sigmas; Mix1 / Mix2 masks differ
    dropped = total = same = 0
    for rnd in range(400):
        m1, m2 = T.edge_mask(0, rnd, 1, 0.1, nbr), T.edge_mask(0, rnd, 2, 0.1, nbr)
        same += m1 == m2
        for m in range(16):
            for j, n in enumerate(nbr[m]):
                if m < n:
                    total += 1
                    dropped += 1 - m1[m][j]
    assert total == 32 * 400
    assert abs(dropped - 0.1 * total) < 4 * math.sqrt(total * 0.1 * 0.9)
    assert same < 40  # P(two independent masks agree) = 0.82^32 ~ 0.2 %


# ------------------------------------------------------------------ consensus distance
def test_consensus_matches_numpy_and_invariances():
    K, P = 5, 1000
    th = _rand(K, P, 9, 0.02)
    s = oracle.consensus_sumsq(th)
    np.testing.assert_allclose(s, ((th - th.mean(0)) ** 2).sum(1), rtol=1e-12)
    np.testing.assert_allclose(oracle.consensus_sumsq(th + 3.25), s, rtol=1e-9)   # translation
    np.testing.assert_allclose(oracle.consensus_sumsq(th[::-1]), s[::-1], rtol=1e-12)  # relabelling
    assert oracle.consensus_sumsq(np.repeat(th[:1], K, 0)).max() < 1e-30  # K=5: the mean of equal values is off by an ulp
    n, q = oracle.cd_finalize(np.array([4.0, 9.0]))
    assert n == 2.5 and q == 6.5


def test_expected_consensus_distance_closed_form():
    """Mix1 = mean, v = 0, iid drift of std sigma: E[CD_sq] = P gamma^2 (1+mu)^2 sigma^2
    (||W2||_F^2 - 1) / K.  K=4 ring, P=2^20, sigma=1e-3 gives 0.154569; the seeded generator
    plus the oracle must land within sampling noise (about 0.2 %)."""
    K, P, sigma = 4, 1 << 20, 1e-3
    tp = gen.theta0(0, K, P)
    tl = gen.local_params(tp, [sigma] * K, 0, 0)
    tn, _ = oracle.outer_round(oracle.dense_W("mean", K), _ring_W(K), tp, tl, np.zeros((K, P)), GAMMA, MU)
    _, cd_sq = oracle.cd_finalize(oracle.consensus_sumsq(tn))
    expect = P * GAMMA ** 2 * (1 + MU) ** 2 * sigma ** 2 * (1.0 / 3.0) / K
    assert expect == pytest.approx(0.154569, rel=1e-5)
    assert cd_sq == pytest.approx(expect, rel=6e-3)


# ------------------------------------------------------------------ variants: subset Mix2, momentum averaging
def test_subset_mix2_limits_and_brute_force():
    K, P = 4, 12
    W1, W2 = oracle.dense_W("mean", K), _ring_W(K)
    tp, tl, v = _rand(K, P, 1, 0.02), _rand(K, P, 2, 0.02), _rand(K, P, 3, 1e-3)
    full = oracle.outer_round(W1, W2, tp, tl, v, GAMMA, MU)
    ident = oracle.outer_round(W1, oracle.dense_W("identity", K), tp, tl, v, GAMMA, MU)
    every = oracle.outer_round_ex(W1, W2, tp, tl, v, GAMMA, MU, mix2_ranges=[(0, P)])
    none = oracle.outer_round_ex(W1, W2, tp, tl, v, GAMMA, MU, mix2_ranges=[(0, 0)])
    assert np.array_equal(every[0], full[0]) and np.array_equal(every[1], full[1])
    assert np.array_equal(none[0], ident[0]) and np.array_equal(none[1], ident[1])
    # columns 4..7 and 10..11 mixed, the rest identity: column by column it is one or the other
    sub = oracle.outer_round_ex(W1, W2, tp, tl, v, GAMMA, MU, mix2_ranges=[(4, 8), (10, 12)])
    for p in range(P):
        src = full if (4 <= p < 8 or p >= 10) else ident
        assert np.array_equal(sub[0][:, p], src[0][:, p]) and np.array_equal(sub[1][:, p], src[1][:, p])


def test_momentum_averaging_reproduces_diloco_trajectory():
    """Mix1 = global average of parameters AND momentum, no Mix2: the averaged model follows
    DiLoCo's trajectory exactly (Sec. 4.2 with the state synchronised as App. B requires):
    x_{r+1} = mean_m z_{m,r+1} = OuterOpt(x_r, -mean_m Delta_{m,r})."""
    K, P, R = 8, 30, 4
    J, I = oracle.dense_W("mean", K), oracle.dense_W("identity", K)
    base = _rand(1, P, 1, 0.02)
    z = np.repeat(base, K, axis=0)
    v = np.zeros((K, P))
    drifts = [_rand(K, P, 20 + r, 1e-3) for r in range(R)]
    means = []
    for r in range(R):
        z, v = oracle.outer_round_ex(J, I, z, z + drifts[r], v, GAMMA, MU, average_momentum=True)
        means.append(z.mean(0))
    ref = _torch_nesterov_steps(base[0], [-drifts[r].mean(0) for r in range(R)])
    for r in range(R):
        np.testing.assert_allclose(means[r], ref[r], rtol=1e-12, atol=1e-16)
    # without the momentum averaging the per-worker states differ, with it Mix1(v) is common
    z2, v2 = oracle.outer_round_ex(J, I, z, z + drifts[0], v, GAMMA, MU, average_momentum=False)
    assert np.abs(v2 - v2.mean(0)).max() > 1e-6
