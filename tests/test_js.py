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


# ------------------------------------------------------------------ GPU parity
@pytest.mark.gpu
@pytest.mark.parametrize("K,U,V,k,shape", [
    (4, 64, 32000, 100, "plain"), (8, 33, 5001, 100, "plain"), (2, 7, 100, 100, "plain"), (3, 5, 70000, 37, "plain"),
    (1, 1, 256, 1, "plain"), (2, 9, 128256, 100, "plain"), (2, 6, 40003, 256, "plain"),
    (8, 33, 5001, 100, "equal_below_cut"),   # many equal logits in the averaged model, below the cut
    (2, 8, 5001, 100, "tie_at_cut"),         # 101 equal logits above everything else: the cut falls inside the group
    (2, 6, 30000, 100, "big_tie_at_cut"),    # 4286 equal top logits: more than the streaming kernel's boundary list holds
    (2, 5, 70000, 100, "ascending"),         # rows in ascending order: the sampling bound is useless, candidates overflow
    (1, 3, 20000, 64, "all_equal"),
    (2, 4, 50001, 100, "descending"),
])
def test_js_distance_gpu(K, U, V, k, shape):
    import torch
    import paper_2606_22768_b200 as fgd
    work, avg = _logits(K, U, V, seed=3)
    if shape == "equal_below_cut":
        avg[:, ::7] = 1.25
    elif shape == "tie_at_cut":
        avg[:, ::50] = 11.0
    elif shape == "big_tie_at_cut":
        avg[:, ::7] = 11.0
    elif shape == "ascending":
        avg = np.sort(avg, axis=1)
    elif shape == "descending":
        avg = np.ascontiguousarray(np.sort(avg, axis=1)[:, ::-1])
    elif shape == "all_equal":
        avg[:] = 0.5
    w = torch.from_numpy(work).cuda()
    a = torch.from_numpy(avg).cuda()
    idx = torch.full((U, k), -1, dtype=torch.int32, device="cuda")
    d = torch.full((K, U), -1.0, dtype=torch.float64, device="cuda")
    cdw = torch.zeros(K, dtype=torch.float64, device="cuda")
    fgd.fgd_js_distance(w, a, idx, d, cdw, top_k=k)
    torch.cuda.synchronize()
    ref_idx, ref_d, ref_cd = ojs.cd_js(work, avg, k)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), ref_idx), "selected tokens must match exactly"
    np.testing.assert_allclose(d.cpu().numpy(), ref_d, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(cdw.cpu().numpy(), ref_d.mean(axis=1), rtol=1e-10, atol=1e-13)
    assert float(cdw.mean()) == pytest.approx(ref_cd, rel=1e-10, abs=1e-13)
    # deterministic
    d2 = torch.zeros_like(d)
    fgd.fgd_js_distance(w, a, idx, d2, cdw, top_k=k)
    torch.cuda.synchronize()
    assert torch.equal(d, d2)


@pytest.mark.gpu
def test_js_distance_argument_errors():
    import torch
    import paper_2606_22768_b200 as fgd
    w = torch.zeros((2, 3, 50), device="cuda"); a = torch.zeros((3, 50), device="cuda")
    idx = torch.zeros((3, 100), dtype=torch.int32, device="cuda")
    d = torch.zeros((2, 3), dtype=torch.float64, device="cuda"); c = torch.zeros(2, dtype=torch.float64, device="cuda")
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_js_distance(w, a, idx, d, c, top_k=100)    # more tokens than the vocabulary has
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
