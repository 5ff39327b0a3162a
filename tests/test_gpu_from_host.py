"""fgd_outer_step_from_host: theta_local streamed from pinned host memory in column chunks.  The
result must be that of the plain call on the whole matrix (bit for bit in theta_new and momentum:
columns are independent) and match the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen
from tests.gpu_util import assert_cd_close, assert_param_close, make_mix, upload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,P,mix1,mix2,chunks,fused", [
    (16, 70001, ("mean",), ("ring",), 8, False),                 # the benchmark's structure, ragged tail
    (8, 5000, ("mean",), ("matching", 0.1), 32, False),          # more chunks than 1024-column blocks
    (16, 40000, ("hypercube", 0.1), ("hypercube", 0.1), 3, True),   # gossip Mix1 gathered in the kernel
    (64, 9000, ("mean",), ("dense", gen.sinkhorn_W(0, 64)), 4, False),   # tensor-core kernel per chunk
    (10, 50003, ("mean",), ("ring", 0.1), 5, False),             # zero-padded onto the 12-worker kernel
    (64, 8000, ("hypercube",), ("ring",), 3, True),              # both mixes as MMAs per chunk
    (64, 6000, ("matching",), ("hypercube",), 2, True),          # one neighbour slot: gathered from the stage
    (4, 3000, ("ring",), ("ring",), 1, False),                   # one chunk, matrix-valued x
])
def test_outer_step_from_host(K, P, mix1, mix2, chunks, fused):
    seed = 9
    ld = P + (4 - P % 4) % 4
    tp = gen.theta0(seed, K, P, 0.02, 5e-4)
    tl = tp + gen.scaled_normal(seed, gen.TENSOR_DRIFT, 0, K, P, np.full(K, 1e-3, np.float32))
    v = gen.scaled_normal(seed, gen.TENSOR_MOMENTUM, 0, K, P, 1e-3)
    d1, W1 = make_mix(mix1, K, 1, seed, 1)
    d2, W2 = make_mix(mix2, K, 1, seed, 2)
    f_tp, g_tp = upload(tp, ld)
    f_v, g_v = upload(v, ld)
    f_tp2, g_tp2 = upload(tp, ld)
    f_v2, g_v2 = upload(v, ld)
    f_tl, _ = upload(tl, ld)
    host_tl = torch.zeros((K, ld), dtype=torch.float32).pin_memory()
    host_tl[:, :P] = torch.from_numpy(tl)
    staging = torch.full((K, ld), -5.0, dtype=torch.float32, device="cuda")
    ctx = fgd.Context(K, P, ld)
    x, vec = None, False
    if not fused:
        vec = mix1[0] == "mean"
        x = torch.empty(P if vec else (K, ld), dtype=torch.float32, device="cuda")
        fgd.fgd_mix(ctx, d1, f_tp, x, out_is_vector=vec)
    m1 = d1 if fused else None
    cd = fgd.fgd_outer_step_from_host(ctx, d2, m1, x, vec, host_tl, staging, f_tp, f_v, f_tp, 0.7, 0.9,
                                      want_cd=True, n_chunks=chunks)
    # the plain call on device-resident inputs
    cd_dev = torch.zeros(K, dtype=torch.float64, device="cuda")
    if not fused:
        fgd.fgd_mix(ctx, d1, f_tp2, x, out_is_vector=vec)
    fgd.fgd_outer_step(ctx, d2, m1, x, vec, f_tl, f_tp2, f_v2, f_tp2, 0.7, 0.9, cd_dev)
    torch.cuda.synchronize()
    assert torch.equal(g_tp, g_tp2) and torch.equal(g_v, g_v2), "chunked and whole-matrix results differ"
    ref_t, ref_v = oracle.outer_round(W1, W2, tp, tl, v, 0.7, 0.9)
    assert_param_close(g_tp, ref_t, "theta_new")
    assert_param_close(g_v, ref_v, "momentum")
    assert_cd_close(cd, oracle.consensus_sumsq(ref_t), P, "chunked consensus sums")
    np.testing.assert_allclose(cd, cd_dev.cpu().numpy(), rtol=1e-6)
    fgd.fgd_device_status(ctx)


def test_from_host_argument_errors():
    K, P = 4, 2048
    ctx = fgd.Context(K, P)
    dev = torch.zeros((K, P), dtype=torch.float32, device="cuda")
    host = torch.zeros((K, P), dtype=torch.float32)
    x = torch.zeros(P, dtype=torch.float32, device="cuda")
    ring = fgd.MixDesc.ring(K)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_outer_step_from_host(ctx, ring, None, x, True, host, dev, dev.clone(), dev.clone(), dev.clone(), n_chunks=0)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError):
        fgd.fgd_outer_step_from_host(ctx, ring, None, x, True, host, dev, dev.clone(), dev.clone(), dev.clone(), n_chunks=33)
    with pytest.raises(TypeError):
        fgd.fgd_outer_step_from_host(ctx, ring, None, x, True, dev, dev, dev.clone(), dev.clone(), dev.clone())
