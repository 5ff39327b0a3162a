"""Oracle-side mixing matrices: topologies, per-round edge failures, renormalisation.

TEST INFRASTRUCTURE ONLY -- plain Python (lists, ints, floats), independent of the
CUDA library's own host builders; neither imports the other.

The paper fixes only that every mixing matrix W_r is symmetric and doubly
stochastic, that global averaging is W = (1/M) 1 1^T, and that "pairwise gossip" is
one random matching whose pairs average (Sec. 3, "Gossip-based Mixing"; App. A,
the table of (Mix1, Mix2) choices).  Its failure model is one sentence: a missed
exchange gives weaker mixing instead of aborting the round (Sec. 1; Sec. 5.2).
Everything else here (ring / hypercube / one-peer schedules, the Bernoulli edge
mask, the two renormalisation rules, the hash) is this build's stated reading:
``edge_mask`` and ``effective_weights`` are PARITY UNPINNED BY THE PAPER (it gives no
formula for either); they are pinned only by what the mathematics fixes -- symmetry,
double stochasticity, the drop rate, the all-alive / all-dead extremes, a hand-worked
fixture -- and by bit-exact agreement with the library's independent implementation.

Sparse form used throughout: ``nbr[m][j]`` = j-th neighbour of worker m or -1 for an
empty slot, ``w[m][j]`` its base weight, ``w_self[m]`` the base self weight.
"""
from __future__ import annotations

import math

MASK64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15

RENORM_NONE = 0
RENORM_SELF_ABSORB = 1
RENORM_METROPOLIS = 2

TAG_MATCHING = 16  # domain tag added to mix_id for the random-matching draws


def mix64(z: int) -> int:
    """The splitmix64 output function (a published 64-bit avalanche mixer)."""
    z &= MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
    return z ^ (z >> 31)


def h64(seed: int, rnd: int, tag: int, a: int, b: int) -> int:
    """Counter-based 64-bit hash of (seed, round, tag, a, b).

    h = mix64(seed + GOLDEN); then for each word x in (round, tag, a, b):
    h = mix64((h XOR x) + GOLDEN).  All arithmetic modulo 2^64.
    """
    h = mix64((seed + GOLDEN) & MASK64)
    for x in (rnd, tag, a, b):
        h = mix64(((h ^ (x & MASK64)) + GOLDEN) & MASK64)
    return h


def is_pow2(k: int) -> bool:
    return k >= 1 and (k & (k - 1)) == 0


def ring(K: int):
    """Ring: neighbours (m-1) mod K, (m+1) mod K in that order, Metropolis weights.

    K >= 3: each edge 1/3, self 1/3.  K == 2: one neighbour, 1/2 and 1/2.  K == 1: W = I.
    """
    if K == 1:
        return [[-1, -1]], [[0.0, 0.0]], [1.0]
    if K == 2:
        return [[1, -1], [0, -1]], [[0.5, 0.0], [0.5, 0.0]], [0.5, 0.5]
    nbr = [[(m - 1) % K, (m + 1) % K] for m in range(K)]
    w = [[1.0 / 3.0, 1.0 / 3.0] for _ in range(K)]
    return nbr, w, [1.0 / 3.0] * K


def onepeer_xor(K: int, rnd: int):
    """One-peer exponential graph: at round r worker m pairs with m XOR 2^(r mod log2 K)."""
    if not is_pow2(K):
        raise ValueError("one-peer XOR schedule needs K a power of two")
    if K == 1:
        return [[-1]], [[0.0]], [1.0]
    bits = K.bit_length() - 1
    j = rnd % bits
    return [[m ^ (1 << j)] for m in range(K)], [[0.5] for _ in range(K)], [0.5] * K


def hypercube(K: int):
    """Static union of the one-peer graphs: neighbours m XOR 2^j, j ascending; weights 1/(1+log2 K)."""
    if not is_pow2(K):
        raise ValueError("hypercube needs K a power of two")
    bits = K.bit_length() - 1
    if bits == 0:
        return [[-1]], [[0.0]], [1.0]
    wt = 1.0 / (1.0 + bits)
    nbr = [[m ^ (1 << j) for j in range(bits)] for m in range(K)]
    return nbr, [[wt] * bits for _ in range(K)], [wt] * K


def random_matching(K: int, seed: int, rnd: int, mix_id: int):
    """Synchronous pairwise random gossip: a random matching, each pair averages.

    Fisher-Yates from the identity permutation: for i = K-1 .. 1,
    j = h64(seed, round, 16 + mix_id, i, 0) mod (i+1), swap pi[i], pi[j].
    Pairs are (pi[0], pi[1]), (pi[2], pi[3]), ...; with odd K pi[K-1] stays alone.
    """
    pi = list(range(K))
    for i in range(K - 1, 0, -1):
        j = h64(seed, rnd, TAG_MATCHING + mix_id, i, 0) % (i + 1)
        pi[i], pi[j] = pi[j], pi[i]
    nbr = [[-1] for _ in range(K)]
    w = [[0.0] for _ in range(K)]
    w_self = [1.0] * K
    for t in range(0, K - 1, 2):
        a, b = pi[t], pi[t + 1]
        nbr[a][0], nbr[b][0] = b, a
        w[a][0] = w[b][0] = 0.5
        w_self[a] = w_self[b] = 0.5
    return nbr, w, w_self


def drop_threshold(p_fail: float) -> int:
    """An edge is dropped iff the top 32 bits of its hash are < floor(p * 2^32) (clamped to [0, 2^32])."""
    if p_fail <= 0.0:
        return 0
    if p_fail >= 1.0:
        return 1 << 32
    return int(math.floor(p_fail * 4294967296.0))


def edge_mask(seed: int, rnd: int, mix_id: int, p_fail: float, nbr):
    """Per-round Bernoulli failure of every UNDIRECTED edge; 1 = alive, 0 = dropped or empty slot.

    Edge {a, b} is keyed by (lo, hi) = (min, max), so both directions agree.
    """
    T = drop_threshold(p_fail)
    mask = []
    for m, row in enumerate(nbr):
        out = []
        for n in row:
            if n < 0:
                out.append(0)
            else:
                lo, hi = (m, n) if m < n else (n, m)
                out.append(0 if (h64(seed, rnd, mix_id, lo, hi) >> 32) < T else 1)
        mask.append(out)
    return mask


def effective_weights(nbr, w, w_self, mask=None, renorm=RENORM_NONE):
    """Weights actually applied this round, in float64.

    An edge is alive iff its slot is non-empty and its mask entry is 1 (mask None = all alive).
    NONE:        dead edges get weight 0, everything else is the base weight.
    SELF_ABSORB: alive edges keep the base weight; each endpoint adds the base weight of
                 its dead edges to its own self weight (what a missed pairwise exchange does).
    METROPOLIS:  with d'_m = number of alive edges at m, every alive edge {m, n} gets
                 1 / (1 + max(d'_m, d'_n)) and the self weight is 1 minus the row's edge weights.
    All three keep a symmetric doubly-stochastic base matrix symmetric; the last two keep
    it doubly stochastic.
    """
    K = len(nbr)
    alive = [[(nbr[m][j] >= 0) and (mask is None or mask[m][j] != 0) for j in range(len(nbr[m]))]
             for m in range(K)]
    deg = [sum(1 for a in alive[m] if a) for m in range(K)]
    w_eff = [[0.0] * len(nbr[m]) for m in range(K)]
    ws_eff = [0.0] * K
    for m in range(K):
        if renorm == RENORM_METROPOLIS:
            tot = 0.0
            for j, n in enumerate(nbr[m]):
                if alive[m][j]:
                    w_eff[m][j] = 1.0 / (1.0 + max(deg[m], deg[n]))
                    tot += w_eff[m][j]
            ws_eff[m] = 1.0 - tot
        else:
            ws = float(w_self[m])
            for j, n in enumerate(nbr[m]):
                if alive[m][j]:
                    w_eff[m][j] = float(w[m][j])
                elif n >= 0 and renorm == RENORM_SELF_ABSORB:
                    ws += float(w[m][j])
            ws_eff[m] = ws
    return w_eff, ws_eff


def dense_from_sparse(nbr, w_eff, ws_eff):
    """Scatter a sparse row description into the dense row-convention matrix W[m][n]."""
    K = len(nbr)
    W = [[0.0] * K for _ in range(K)]
    for m in range(K):
        W[m][m] += ws_eff[m]
        for j, n in enumerate(nbr[m]):
            if n >= 0:
                W[m][n] += w_eff[m][j]
    return W


def mean_matrix(K: int):
    """Global averaging, W = (1/K) 1 1^T (Sec. 3)."""
    return [[1.0 / K] * K for _ in range(K)]


def identity_matrix(K: int):
    return [[1.0 if m == n else 0.0 for n in range(K)] for m in range(K)]
