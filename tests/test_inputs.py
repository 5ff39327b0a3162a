"""The seeded input generator: distribution sanity on CPU, and the CUDA twin gives the same bits."""
import numpy as np
import pytest

from fgd_inputs import gen


def test_std_normal_moments_and_reproducibility():
    e = gen.std_normal(0, gen.TENSOR_DRIFT, 3, 5, 0, 1 << 20)
    assert e.dtype == np.float32
    assert abs(float(e.mean())) < 4e-3 and abs(float(e.var()) - 1.0) < 5e-3
    assert 2.6 < float((e.astype(np.float64) ** 4).mean()) < 3.0   # Irwin-Hall(8): kurtosis 2.85
    assert np.array_equal(e[1000:2000], gen.std_normal(0, gen.TENSOR_DRIFT, 3, 5, 1000, 2000))
    assert not np.array_equal(e[:100], gen.std_normal(0, gen.TENSOR_DRIFT, 4, 5, 0, 100))
    assert not np.array_equal(e[:100], gen.std_normal(1, gen.TENSOR_DRIFT, 3, 5, 0, 100))


def test_theta0_rows_identical_unless_offset():
    a = gen.theta0(0, 4, 1000)
    assert np.array_equal(a[0], a[3]) and abs(float(a.std()) - 0.02) < 2e-3
    b = gen.theta0(0, 4, 1000, worker_std=5e-4)
    assert not np.array_equal(b[0], b[3])
    assert np.array_equal(gen.theta0(0, 4, 1000, p0=100, p1=200), a[:, 100:200])


def test_sigmas_and_sinkhorn():
    s = gen.drift_sigmas(0, 16, 5e-4, 2e-3)
    assert s.dtype == np.float32 and (s >= 5e-4).all() and (s < 2e-3).all() and len(set(s.tolist())) == 16
    W = gen.sinkhorn_W(0, 64)
    assert W.dtype == np.float32 and np.array_equal(W, W.T) and (W > 0).all()
    W64 = W.astype(np.float64)
    assert np.abs(W64.sum(0) - 1).max() < 64 * 1e-7 and np.abs(W64.sum(1) - 1).max() < 64 * 1e-7


@pytest.mark.gpu
def test_cuda_twin_same_bits():
    import torch
    from fgd_inputs import gpu
    K, P, ld = 5, 100003, 100008
    full = torch.full((K, ld), -777.0, dtype=torch.float32, device="cuda")
    gpu.theta0(full[:, :P], 3, 0.02, 5e-4)
    ref = gen.theta0(3, K, P, 0.02, 5e-4)
    assert np.array_equal(full[:, :P].cpu().numpy(), ref)
    sig = gen.drift_sigmas(3, K, 5e-4, 2e-3)
    loc = torch.full((K, ld), -777.0, dtype=torch.float32, device="cuda")
    for rnd in (0, 7):
        gpu.local_steps(loc[:, :P], full[:, :P], sig, 3, rnd)
        assert np.array_equal(loc[:, :P].cpu().numpy(), gen.local_params(ref, sig, 3, rnd))
    assert bool((loc[:, P:] == -777.0).all())
    # a column block regenerated on the CPU matches the same block of the GPU tensor
    blk = gen.local_params(ref[:, 5000:6000], sig, 3, 7, p0=5000)
    assert np.array_equal(loc[:, 5000:6000].cpu().numpy(), blk)
