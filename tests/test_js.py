"""JS functional-disagreement metric: oracle pins (CPU) and GPU parity."""
import numpy as np
import pytest

from oracle import js as ojs
from fgd_inputs import gen


def _logits(K, U, V, seed=0, spread=2.0, noise=0.3):
    avg = gen.scaled_normal(seed, gen.TENSOR_AUX, 0, U, V, spread)            # [U, V]
    work = np.stack([avg + gen.scaled_normal(seed, gen.TENSOR_AUX, 1 + m, U, V, noise) for m in range(K)])
    return work.astype(np.float32), avg.astype(np.float32)


# ------------------------------------------------------------------ oracle pins
def test_js_matches_scipy_and_bounds():
    from scipy.spatial.distance import jensenshannon
    from scipy.special import softmax
    rng = np.random.default_rng(0)
    for _ in range(20):
        a, b = rng.normal(0, 3, 50), rng.normal(0, 3, 50)
        ours = ojs.js_distance(a, b)
        ref = jensenshannon(softmax(a), softmax(b), base=2.0)    # sqrt(JS / ln 2)
        assert ours == pytest.approx(ref, rel=1e-10, abs=1e-14)
        assert 0.0 <= ours <= 1.0
        assert ours == pytest.approx(ojs.js_distance(b, a), rel=1e-12)
    assert ojs.js_distance(a, a) == 0.0
    assert ojs.js_distance(a, a + 7.5) == pytest.approx(0.0, abs=1e-7)     # softmax is shift invariant
    # disjoint supports: the distance reaches its maximum 1
    p = np.array([0.0, 0.0, -1e4, -1e4]); q = np.array([-1e4, -1e4, 0.0, 0.0])
    assert ojs.js_distance(p, q) == pytest.approx(1.0, abs=1e-12)
    # two-point closed form: p = (1, 0), q = (1/2, 1/2): JS = 1/2 ln(4/3) + 1/4 ln(2/3) + 1/4 ln 2
    js = 0.5 * np.log(4 / 3) + 0.25 * np.log(2 / 3) + 0.25 * np.log(2.0)
    assert ojs.js_distance(np.array([0.0, -1e4]), np.array([0.0, 0.0])) == pytest.approx(np.sqrt(js / np.log(2)), rel=1e-12)


def test_top_tokens_and_truncated_metric():
    row = np.array([0.1, 5.0, 3.0, 5.0, -2.0, 3.0, 4.0])
    assert ojs.top_tokens(row, 3).tolist() == [1, 3, 6]
    assert ojs.top_tokens(row, 4).tolist() == [1, 2, 3, 6]          # tie at 3.0 -> the lower index
    K, U, V, k = 3, 5, 400, 100
    work, avg = _logits(K, U, V, seed=1)
    idx, d, cd = ojs.cd_js(work, avg, k)
    assert idx.shape == (U, k) and d.shape == (K, U)
    from scipy.spatial.distance import jensenshannon
    from scipy.special import softmax
    for u in range(U):
        keep = np.argsort(-avg[u].astype(np.float64), kind="stable")[:k]
        assert set(idx[u].tolist()) == set(keep.tolist())
        for m in range(K):
            ref = jensenshannon(softmax(work[m, u, idx[u]].astype(np.float64)), softmax(avg[u, idx[u]].astype(np.float64)), base=2.0)
            assert d[m, u] == pytest.approx(ref, rel=1e-9)
    assert cd == pytest.approx(d.mean())
    # identical workers and average: zero disagreement
    _, d0, cd0 = ojs.cd_js(np.stack([avg, avg]), avg, k)
    assert cd0 == 0.0 and d0.max() == 0.0
