"""GPU parity: every C-ABI entry point against the float64 oracle on the same seeded inputs.

Bar: indices and edge masks bit-exact (checked in make_mix), fp32 parameters within max relative
error 1e-5 (absolute 1e-7 near zero), consensus sums within relative 1e-5.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen
from tests.gpu_util import (Scenario, assert_cd_close, assert_param_close, check_padding, make_mix,
                            padded, upload)

pytestmark = pytest.mark.gpu

SINK64 = gen.sinkhorn_W(0, 64)
PATHS = [pytest.param(fgd.FGD_PATH_AUTO, id="auto"), pytest.param(fgd.FGD_PATH_TMA, id="tma"),
         pytest.param(fgd.FGD_PATH_REGISTER, id="reg"), pytest.param(fgd.FGD_PATH_TMA_FP32, id="tma_fp32")]


def _inputs(K, P, seed=0, worker_std=5e-4, sigma=1e-3):
    tp = gen.theta0(seed, K, P, 0.02, worker_std)
    tl = gen.local_params(tp, [sigma] * K, seed, 0)
    v = gen.scaled_normal(seed, gen.TENSOR_MOMENTUM, 0, K, P, 1e-3)
    return tp, tl, v


# ------------------------------------------------------------------ fgd_outer_grad
@pytest.mark.parametrize("K,P,ld", [(4, 1 << 20, None), (16, 100003, 100003), (3, 4100, 4352), (1, 1, 1), (64, 777, 780)])
def test_outer_grad(K, P, ld):
    ld = P if ld is None else ld
    tp, tl, _ = _inputs(K, P)
    f_tp, _ = upload(tp, ld)
    f_tl, _ = upload(tl, ld)
    f_g, g = padded(K, P, ld)
    ctx = fgd.Context(K, P, ld)
    fgd.fgd_outer_grad(ctx, f_tp, f_tl, f_g)
    torch.cuda.synchronize()
    ref = oracle.outer_grad(tp, tl)
    # a single fp32 subtraction of fp32 inputs is correctly rounded: must equal the rounded oracle
    assert np.array_equal(g.cpu().numpy(), ref.astype(np.float32))
    check_padding(f_g, P, "g")
    assert ctx.launch_count == 1


# ------------------------------------------------------------------ fgd_mix
MIX_CASES = [
    (4, 1 << 18, ("mean",)), (4, 70001, ("ring",)), (8, 50000, ("xor",)), (16, 33333, ("hypercube",)),
    (16, 40960, ("hypercube", 0.3)), (16, 5000, ("ring", 0.2, fgd.FGD_RENORM_SELF_ABSORB)),
    (16, 20000, ("matching",)), (9, 3000, ("matching",)), (5, 12345, ("ring",)), (3, 999, ("mean",)),
    (32, 20002, ("hypercube", 0.1)), (64, 10000, ("dense", SINK64)), (64, 4097, ("ring",)),
    (16, 8192, ("dense", gen.sinkhorn_W(1, 16))), (7, 2048, ("dense", gen.sinkhorn_W(2, 7))),
    (2, 1000, ("ring",)), (1, 100, ("identity",)), (8, 1000, ("identity",)),
    (64, 70004, ("mean",)), (32, 50000, ("mean",)), (64, 30001, ("mean",)),   # threads share a column (and its fall-back)
    # tensor-core mix: worker counts 17..64 (zero-padded to 32 / 48 / 64), sparse mixes densified
    (48, 9001, ("ring",)), (40, 5000, ("dense", gen.sinkhorn_W(8, 40))), (33, 4100, ("matching",)), (63, 3000, ("mean",)),
    (32, 6002, ("dense", gen.sinkhorn_W(7, 32))), (24, 7000, ("ring", 0.3)), (17, 2000, ("dense", gen.sinkhorn_W(9, 17))),
    (64, 20000, ("hypercube", 0.1)), (8, 30000, ("hypercube", 0.2)), (16, 9000, ("randgraph", 5, 0.2)), (40, 3000, ("randgraph", 3)), (7, 2000, ("randgraph", 2)),
    # sparse mixes above 16 workers: the TMA-pipelined row gather (run-time worker and slot counts, ragged tails)
    (17, 1001, ("ring",)), (23, 70003, ("matching",)), (31, 5000, ("circulant", 2)), (32, 9999, ("circulant", 3, 0.2)),
    (47, 3000, ("randgraph", 8)), (57, 130, ("ring", 0.3)), (63, 20001, ("randgraph", 5, 0.2)), (64, 127, ("matching",)),
    (20, 4096, ("identity",)),
    # every worker count up to 16 that is not a power of two has stand-alone kernels of its own
    (3, 5001, ("ring",)), (6, 4100, ("matching",)), (6, 70001, ("ring", 0.2)), (7, 9000, ("ring",)), (10, 6000, ("randgraph", 3)),
    (11, 3001, ("ring", 0.3, fgd.FGD_RENORM_SELF_ABSORB)), (12, 8000, ("matching",)), (13, 5000, ("randgraph", 5)),
    (14, 4000, ("ring",)), (15, 7001, ("mean",)), (10, 2000, ("mean",)), (12, 3000, ("randgraph", 1)),
]


@pytest.mark.parametrize("K,P,spec", MIX_CASES)
def test_mix_matrix_output(K, P, spec):
    x = gen.theta0(3, K, P, 0.02, 5e-3)
    desc, W = make_mix(spec, K, 1, 3, 1)
    ld = P + (4 - P % 4) % 4 + 4
    f_in, _ = upload(x, ld)
    f_out, out = padded(K, P, ld)
    ctx = fgd.Context(K, P, ld)
    fgd.fgd_mix(ctx, desc, f_in, f_out)
    torch.cuda.synchronize()
    assert_param_close(out, oracle.mix(W, x), f"mix {spec[0]} K={K}")
    check_padding(f_out, P, "mix out")
    # in place gives the same bits
    fgd.fgd_mix(ctx, desc, f_in, f_in)
    torch.cuda.synchronize()
    assert torch.equal(f_in[:, :P], out)


@pytest.mark.parametrize("K,P", [(4, 1 << 20), (16, 30001), (6, 513), (64, 4096), (64, 100004), (32, 65540), (32, 999),
                                 (6, 5120), (13, 40004), (11, 1000)])
def test_mix_mean_vector_output(K, P):
    x = gen.theta0(4, K, P, 0.02, 5e-3)
    f_in, _ = upload(x, P)
    out = torch.full((P + 8,), -777.0, dtype=torch.float32, device="cuda")
    ctx = fgd.Context(K, P)
    fgd.fgd_mix(ctx, fgd.MixDesc.mean(K), f_in, out, out_is_vector=True)
    torch.cuda.synchronize()
    assert_param_close(out[:P], oracle.mix(oracle.dense_W("mean", K), x)[0], "mean vector")
    assert bool((out[P:] == -777.0).all())


# ------------------------------------------------------------------ fgd_consensus_distance
@pytest.mark.parametrize("K,P,ld", [(4, 1 << 20, None), (16, 100001, 100004), (64, 20000, 20000), (32, 30002, 30002),
                                     (5, 7777, 7780), (1, 50, 50), (2, 3, 4), (64, 150004, 150016), (32, 200000, 200000),
                                     (64, 131, 132), (32, 4, 4)]
                         + [(K, 20000 + 37 * K, 20000 + 37 * K + (4 - (37 * K) % 4) % 4) for K in (3, 6, 7, 9, 10, 11, 12, 13, 14, 15)]
                         + [(13, 5001, 5001)]       # odd row stride: the run-time-K kernel
                         # 17-31 / 33-63 workers on the 32- / 64-worker split kernels with the rows beyond K left out
                         + [(17, 30001, 30004), (24, 4096, 4096), (31, 70003, 70004), (33, 20002, 20004), (47, 9000, 9000),
                            (56, 131, 132), (63, 50001, 50004), (40, 3, 4), (23, 20001, 20001)])
def test_consensus_distance(K, P, ld):
    ld = P if ld is None else ld
    th = gen.theta0(5, K, P, 0.02, 7e-4)
    f_th, _ = upload(th, ld)
    s = torch.full((K,), -1.0, dtype=torch.float64, device="cuda")
    ctx = fgd.Context(K, P, ld)
    fgd.fgd_consensus_distance(ctx, f_th, s)
    torch.cuda.synchronize()
    ref = oracle.consensus_sumsq(th)
    assert_cd_close(s, ref, P, "consensus")
    got = fgd.fgd_cd_finalize(s.cpu().numpy())
    exp = oracle.cd_finalize(ref)
    assert got[0] == pytest.approx(exp[0], rel=1e-5, abs=1e-9) and got[1] == pytest.approx(exp[1], rel=1e-5, abs=1e-12)
    # deterministic: a second call gives the same bits
    s2 = torch.zeros_like(s)
    fgd.fgd_consensus_distance(ctx, f_th, s2)
    torch.cuda.synchronize()
    assert torch.equal(s, s2)


# ------------------------------------------------------------------ fgd_outer_step, single call
STEP_CASES = [
    # K, P, mix1, mix2
    (4, 1 << 18, ("mean",), ("ring",)),
    (8, 60001, ("mean",), ("xor",)),
    (16, 50000, ("mean",), ("ring",)),
    (16, 30003, ("hypercube", 0.2), ("hypercube", 0.2)),
    (16, 20000, ("matching",), ("matching",)),
    (16, 8000, ("identity",), ("mean",)),
    (16, 8000, ("mean",), ("identity",)),
    (64, 9000, ("mean",), ("dense", SINK64)),
    (64, 4100, ("mean",), ("hypercube",)),
    (32, 10002, ("ring",), ("ring", 0.3)),
    (16, 6000, ("mean",), ("dense", gen.sinkhorn_W(1, 16))),
    (6, 5001, ("ring",), ("dense", gen.sinkhorn_W(2, 6))),
    (5, 3000, ("mean",), ("ring",)),
    (3, 2000, ("matching",), ("mean",)),
    (2, 1000, ("mean",), ("ring",)),
    (1, 300, ("identity",), ("identity",)),
    # degenerate / extreme descriptors
    (16, 12000, ("mean",), ("circulant", 4)),                                   # FGD_MAX_D = 8 neighbour slots
    (16, 9000, ("circulant", 4, 0.3), ("circulant", 4, 0.3)),                   # ... with failures, both mixes
    (8, 5000, ("mean",), ("isolated",)),                                        # D = 0
    (16, 7000, ("mean",), ("hypercube", 1.0)),                                  # every edge dropped: Mix2 = identity
    (16, 7000, ("mean",), ("hypercube", 0.4, fgd.FGD_RENORM_NONE)),             # no renormalisation: rows sum to < 1
    (16, 7000, ("ring", 0.5, fgd.FGD_RENORM_SELF_ABSORB), ("ring", 0.5, fgd.FGD_RENORM_SELF_ABSORB)),
    # worker counts between the compile-time kernels: zero-padded onto the 64-worker tensor-core kernel
    (48, 9001, ("mean",), ("dense", gen.sinkhorn_W(3, 48))),
    (48, 5000, ("ring",), ("ring", 0.2)),
    (63, 4100, ("mean",), ("dense", gen.sinkhorn_W(4, 63))),
    (33, 4099, ("ring",), ("matching",)),
    (24, 7000, ("mean",), ("dense", gen.sinkhorn_W(5, 24))),
    (17, 6002, ("matching",), ("ring",)),
    (40, 3000, ("mean",), ("mean",)),
    # worker counts zero-padded onto the 6, 8, 12 and 16-worker fp32 kernels (5; 7; 9-11; 13-15)
    (5, 70001, ("mean",), ("ring",)),
    (5, 9000, ("ring", 0.2), ("ring", 0.2)),
    (7, 40002, ("mean",), ("dense", gen.sinkhorn_W(2, 7))),
    (7, 30000, ("matching",), ("randgraph", 3, 0.2)),
    (9, 30001, ("ring",), ("ring",)),
    (10, 50003, ("mean",), ("randgraph", 5)),
    (11, 20000, ("randgraph", 4, 0.1), ("circulant", 3)),
    (13, 40001, ("mean",), ("dense", gen.sinkhorn_W(6, 13))),
    (14, 30002, ("circulant", 2, 0.2), ("circulant", 2, 0.2)),
    (15, 60000, ("mean",), ("circulant", 4)),
    (15, 3, ("ring",), ("ring",)),
    # gossip Mix1 fused into the tensor-core kernel (gathered from the staged theta_prev)
    (64, 5001, ("hypercube", 0.1), ("hypercube", 0.1)),
    (64, 4000, ("ring",), ("dense", SINK64)),
    (64, 3000, ("identity",), ("ring",)),
    (32, 6000, ("matching",), ("dense", gen.sinkhorn_W(7, 32))),
    (56, 3001, ("circulant", 4, 0.2), ("circulant", 3)),
    # three neighbour slots run as the compile-time four; five at K = 32 go to the tensor-core kernel
    (8, 9000, ("hypercube", 0.2), ("hypercube",)),
    (8, 5001, ("mean",), ("hypercube", 0.3)),
    (32, 7000, ("hypercube",), ("hypercube", 0.1)),
    (32, 4001, ("mean",), ("hypercube",)),
    # the row-gather kernel (fused gossip Mix1 or matrix x at 17-28 and 33-64 workers): fewer columns than a tile,
    # ragged tails, one to eight neighbour slots, both CTA shapes
    (40, 3, ("ring",), ("ring",)),
    (24, 130, ("matching",), ("ring", 0.3)),
    (64, 127, ("ring",), ("circulant", 2)),
    (28, 4100, ("randgraph", 3), ("randgraph", 5)),
    (33, 5000, ("circulant", 4, 0.2), ("circulant", 4)),
    (21, 9001, ("identity",), ("ring",)),
    (17, 70002, ("matching", 0.2), ("matching",)),
    (63, 8000, ("randgraph", 8, 0.1), ("ring",)),
    # fewer columns than one tile (and than one vector)
    (64, 5, ("mean",), ("dense", SINK64)),
    (48, 1, ("mean",), ("ring",)),
    (16, 3, ("mean",), ("ring",)),
    (8, 130, ("ring",), ("xor",)),
    (3, 2, ("mean",), ("ring",)),
    # irregular graphs: uneven degrees, empty slots, odd slot counts
    (12, 5000, ("randgraph", 3), ("randgraph", 5, 0.2)),
    (16, 6001, ("randgraph", 5, 0.1), ("randgraph", 3)),
    (48, 4000, ("randgraph", 7), ("randgraph", 7, 0.3)),
    (64, 3000, ("randgraph", 3, 0.2), ("randgraph", 6)),
]


@pytest.mark.parametrize("K,P,mix1,mix2", STEP_CASES)
@pytest.mark.parametrize("mode", ["x_given", "mix1_fused"])
@pytest.mark.parametrize("path", PATHS)
def test_outer_step_single_call(K, P, mix1, mix2, mode, path):
    if mode == "x_given" and mix1[0] == "identity":
        pytest.skip("identity Mix1 has no transfer")
    if mode == "mix1_fused" and mix1[0] == "dense":
        pytest.skip("dense Mix1 is not fused")
    tp, tl, v = _inputs(K, P, seed=7)
    d1, W1 = make_mix(mix1, K, 2, 7, 1)
    d2, W2 = make_mix(mix2, K, 2, 7, 2)
    ld = P + (4 - P % 4) % 4
    f_tp, g_tp = upload(tp, ld)
    f_tl, _ = upload(tl, ld)
    f_v, g_v = upload(v, ld)
    f_new, g_new = padded(K, P, ld)
    cd = torch.zeros(K, dtype=torch.float64, device="cuda")
    ctx = fgd.Context(K, P, ld)
    fgd.fgd_set_path(ctx, path)
    if mode == "x_given":
        vec = mix1[0] == "mean"
        x = torch.empty(P if vec else (K, ld), dtype=torch.float32, device="cuda")
        fgd.fgd_mix(ctx, d1, f_tp, x, out_is_vector=vec)
    try:
        if mode == "x_given":
            fgd.fgd_outer_step(ctx, d2, None, x, vec, f_tl, f_tp, f_v, f_new, 0.7, 0.9, cd)
        else:
            fgd.fgd_outer_step(ctx, d2, d1, None, False, f_tl, f_tp, f_v, f_new, 0.7, 0.9, cd)
    except fgd.FgdError as e:
        # a FORCED fp32 pipeline must refuse, not fall back, when two of its stages do not fit in
        # shared memory (63 workers; 56 or 64 with a staged matrix-valued x)
        if path == fgd.FGD_PATH_TMA_FP32 and K > 48 and e.status == fgd.FGD_ERR_UNSUPPORTED:
            return
        raise
    torch.cuda.synchronize()
    ref_t, ref_v = oracle.outer_round(W1, W2, tp, tl, v, 0.7, 0.9)
    assert_param_close(g_new, ref_t, "theta_new")
    assert_param_close(g_v, ref_v, "momentum")
    assert_cd_close(cd, oracle.consensus_sumsq(ref_t), P, "fused cd")
    assert torch.equal(g_tp.cpu(), torch.from_numpy(tp)), "theta_prev must not change out of place"
    for full, name in ((f_new, "theta_new"), (f_v, "momentum")):
        check_padding(full, P, name)
    # in place (theta_new == theta_prev), no consensus output: same bits as out of place
    f_v2, g_v2 = upload(v, ld)
    if mode == "x_given":
        fgd.fgd_outer_step(ctx, d2, None, x, vec, f_tl, f_tp, f_v2, f_tp, 0.7, 0.9, None)
    else:
        fgd.fgd_outer_step(ctx, d2, d1, None, False, f_tl, f_tp, f_v2, f_tp, 0.7, 0.9, None)
    torch.cuda.synchronize()
    assert torch.equal(g_tp, g_new) and torch.equal(g_v2, g_v)
    fgd.fgd_device_status(ctx)


def test_outer_step_unaligned_pointers_take_the_elementwise_path():
    K, P = 16, 5003
    tp, tl, v = _inputs(K, P, seed=9)
    d1, W1 = make_mix(("mean",), K, 0, 9, 1)
    d2, W2 = make_mix(("ring",), K, 0, 9, 2)
    ld = P + 2
    bufs = [torch.full((K * ld + 1,), -777.0, dtype=torch.float32, device="cuda") for _ in range(4)]
    views = [b[1:].view(K, ld) for b in bufs]  # base pointer 4 bytes off a 16-byte boundary
    for view, a in zip(views[:3], (tp, tl, v)):
        view[:, :P].copy_(torch.from_numpy(a))
    ctx = fgd.Context(K, P, ld)
    fgd.fgd_set_path(ctx, fgd.FGD_PATH_TMA)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_outer_step(ctx, d2, d1, None, False, views[1], views[0], views[2], views[3], 0.7, 0.9, None)
    assert e.value.status == fgd.FGD_ERR_UNSUPPORTED
    fgd.fgd_set_path(ctx, fgd.FGD_PATH_AUTO)
    fgd.fgd_outer_step(ctx, d2, d1, None, False, views[1], views[0], views[2], views[3], 0.7, 0.9, None)
    torch.cuda.synchronize()
    ref_t, ref_v = oracle.outer_round(W1, W2, tp, tl, v, 0.7, 0.9)
    assert_param_close(views[3][:, :P], ref_t, "theta_new")
    assert_param_close(views[2][:, :P], ref_v, "momentum")
    assert bool((views[3][:, P:] == -777.0).all()) and float(bufs[3][0]) == -777.0


def test_lr_mu_are_honoured():
    K, P = 4, 4096
    tp, tl, v = _inputs(K, P, seed=11)
    d1, W1 = make_mix(("ring",), K, 0, 11, 1)
    d2, W2 = make_mix(("mean",), K, 0, 11, 2)
    for lr, mu in ((1.0, 0.0), (0.3, 0.5)):
        f_tp, _ = upload(tp, P)
        f_tl, _ = upload(tl, P)
        f_v, g_v = upload(v, P)
        f_new, g_new = padded(K, P, P)
        fgd.fgd_outer_step(fgd.Context(K, P), d2, d1, None, False, f_tl, f_tp, f_v, f_new, lr, mu, None)
        torch.cuda.synchronize()
        ref_t, ref_v = oracle.outer_round(W1, W2, tp, tl, v, lr, mu)
        assert_param_close(g_new, ref_t, f"theta_new lr={lr}")
        assert_param_close(g_v, ref_v, f"momentum mu={mu}")


# ------------------------------------------------------------------ multi-round scenarios (the configs, reduced P)
@pytest.mark.parametrize("path", PATHS)
def test_config1_full_size(path):
    """K=4, P=2^20, Mix1 mean, Mix2 ring 1/3, one round, seed 0 -- every element compared."""
    Scenario(4, 1 << 20, ("mean",), ("ring",), seed=0, path=path).run(1)
    Scenario(4, 1 << 20, ("mean",), ("ring",), seed=0, worker_std=5e-4, mode="fused", path=path).run(1)


@pytest.mark.parametrize("path", PATHS)
def test_config2_reduced(path):
    """K=8, one-peer XOR Mix2 over 10 rounds (P reduced to 2^17+37, ragged)."""
    Scenario(8, (1 << 17) + 37, ("mean",), ("xor",), ld=(1 << 17) + 40, seed=0, path=path).run(10)


@pytest.mark.parametrize("path", PATHS)
def test_config3_reduced(path):
    """K=16, per-worker drift scale U[5e-4, 2e-3], side-stream Mix1 mean, ring Mix2, 10 rounds."""
    sig = gen.drift_sigmas(0, 16, 5e-4, 2e-3)
    Scenario(16, 150000, ("mean",), ("ring",), seed=0, sigmas=sig, path=path).run(10)


@pytest.mark.parametrize("mode", ["factored", "fused"])
@pytest.mark.parametrize("path", PATHS)
def test_config4_reduced(mode, path):
    """K=16 hypercube gossip for both mixes, independent p=0.1 edge failures, Metropolis
    renormalisation, 20 rounds, consensus distance every round."""
    Scenario(16, 65536 + 12, ("hypercube", 0.1), ("hypercube", 0.1), seed=0, mode=mode, path=path).run(20)


@pytest.mark.parametrize("path", PATHS)
def test_config5_reduced(path):
    """K=64 dense Sinkhorn Mix2, Mix1 mean, 5 rounds."""
    Scenario(64, 40000, ("mean",), ("dense", SINK64), seed=0, path=path).run(5)


def test_pairwise_gossip_presets():
    """The paper's four (Mix1, Mix2) presets with random-matching pairwise gossip, 4 rounds each."""
    for m1, m2 in ((("identity",), ("mean",)), (("matching",), ("matching",)), (("mean",), ("identity",)),
                   (("mean",), ("matching",))):
        Scenario(8, 20001, m1, m2, ld=20004, seed=3, in_place=False).run(4)


def test_diloco_preset_reaches_exact_consensus():
    s = Scenario(16, 30000, ("identity",), ("mean",), seed=1).run(3)
    rows = s.g_new
    assert torch.equal(rows[0], rows[7]) and torch.equal(rows[0], rows[15])
    assert float(s.drv.cd_sumsq.max()) <= 1e-12 * 30000


def test_nonzero_initial_momentum_and_odd_K():
    Scenario(7, 9999, ("ring", 0.2), ("ring", 0.2), ld=10000, seed=5, v0_std=1e-3, worker_std=1e-3).run(3)
    Scenario(32, 12346, ("mean",), ("hypercube", 0.05), seed=6, v0_std=1e-3).run(3)


# ------------------------------------------------------------------ the paper's variants: -subset and GlobalM1S
def _subset(P):
    """About 43 % of the columns in three blocks (embeddings, LM head, first layers), on 4-column bounds."""
    a, b, c = int(0.18 * P) // 4 * 4, int(0.55 * P) // 4 * 4, int(0.80 * P) // 4 * 4
    return [(0, a), (b, c - (c - b) // 3 // 4 * 4), (c, P)]


VARIANTS = [
    # name, K, P, mix1, mix2, subset?, average momentum?
    ("GlobalM1LocalM2-subset", 8, 40004, ("mean",), ("matching",), True, False),
    ("GlobalM1S", 8, 30000, ("mean",), ("identity",), False, True),
    ("GlobalM1SLocalM2", 16, 30001, ("mean",), ("matching",), False, True),
    ("GlobalM1SLocalM2-subset", 16, 50000, ("mean",), ("matching",), True, True),
    ("ring-subset-runtimeK", 6, 9000, ("mean",), ("ring",), True, True),
    ("dense-subset", 64, 6000, ("mean",), ("dense", SINK64), True, False),
    ("dense-GlobalM1S", 64, 5000, ("mean",), ("dense", SINK64), False, True),
    ("dense16-subset", 16, 8000, ("ring",), ("dense", gen.sinkhorn_W(1, 16)), True, False),
    ("dense48-GlobalM1S", 48, 5000, ("mean",), ("dense", gen.sinkhorn_W(3, 48)), False, True),
    ("ring40-GlobalM1S", 40, 4001, ("mean",), ("ring",), False, True),
    ("dense48-subset", 48, 6000, ("mean",), ("dense", gen.sinkhorn_W(3, 48)), True, False),
    ("ring24-subset-GlobalM1S", 24, 9000, ("mean",), ("ring",), True, True),
    ("ring13-subset-GlobalM1S-padded", 13, 30000, ("mean",), ("ring",), True, True),
    ("dense10-subset-padded", 10, 20000, ("mean",), ("dense", gen.sinkhorn_W(8, 10)), True, False),
]


@pytest.mark.parametrize("name,K,P,mix1,mix2,subset,avg", VARIANTS, ids=[v[0] for v in VARIANTS])
@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", ["factored", "fused"])
def test_paper_variants(name, K, P, mix1, mix2, subset, avg, path, mode):
    ld = P + (4 - P % 4) % 4
    Scenario(K, P, mix1, mix2, ld=ld, seed=4, v0_std=1e-3, worker_std=5e-4, mode=mode, path=path,
             mix2_ranges=_subset(P) if subset else None, average_momentum=avg).run(3)


@pytest.mark.parametrize("K,P,mix2", [(16, 50001, ("ring",)), (8, 30000, ("xor",)), (64, 9000, ("dense", SINK64)),
                                       (64, 5000, ("hypercube",)), (6, 7000, ("ring",)), (2, 4000, ("ring",)),
                                       (48, 6001, ("ring",)), (20, 5000, ("dense", gen.sinkhorn_W(6, 20))),
                                       (13, 30001, ("ring",)), (10, 20000, ("randgraph", 3))])   # zero-padded fp32 shapes
@pytest.mark.parametrize("path", PATHS)
def test_step_emits_next_rounds_global_average(K, P, mix2, path):
    """Mix1 = global average chained through the fused step: round r writes x_{r+1} = mean(theta_new),
    round r+1 reads it instead of running a Mix1 kernel.  Same values as Algorithm 1."""
    ld = P + (4 - P % 4) % 4
    Scenario(K, P, ("mean",), mix2, ld=ld, seed=8, path=path, chain_mix1=True, v0_std=1e-3).run(4)


def test_variant_argument_errors():
    K, P = 4, 1024
    ctx = fgd.Context(K, P)
    a = torch.zeros((K, P), device="cuda")
    b, c, d = torch.zeros_like(a), torch.zeros_like(a), torch.zeros_like(a)
    ring, mean = fgd.MixDesc.ring(K), fgd.MixDesc.mean(K)
    with pytest.raises(fgd.FgdError) as e:    # range bounds must be multiples of 4 columns
        fgd.fgd_outer_step_ex(ctx, ring, mean, None, False, b, a, c, d, mix2_ranges=[(2, 8)])
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError) as e:    # beyond P
        fgd.fgd_outer_step_ex(ctx, ring, mean, None, False, b, a, c, d, mix2_ranges=[(0, P + 4)])
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError) as e:    # too many ranges
        fgd.fgd_outer_step_ex(ctx, ring, mean, None, False, b, a, c, d, mix2_ranges=[(4 * i, 4 * i + 4) for i in range(9)])
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError) as e:    # x_next may not be the x this call reads
        xv = torch.zeros(P, device="cuda")
        fgd.fgd_outer_step_ex(ctx, ring, None, xv, True, b, a, c, d, x_next=xv)
    assert e.value.status == fgd.FGD_ERR_ALIAS
    with pytest.raises(fgd.FgdError) as e:    # momentum averaging belongs to a global Mix1
        fgd.fgd_outer_step_ex(ctx, ring, ring, None, False, b, a, c, d, average_momentum=True)
    assert e.value.status == fgd.FGD_ERR_UNSUPPORTED


# ------------------------------------------------------------------ determinism, errors
def test_outer_step_is_bitwise_deterministic():
    K, P = 16, 200000
    tp, tl, v = _inputs(K, P, seed=2)
    d2, _ = make_mix(("hypercube", 0.1), K, 0, 2, 2)
    outs = []
    for _ in range(2):
        f_tp, _ = upload(tp, P)
        f_tl, _ = upload(tl, P)
        f_v, _ = upload(v, P)
        cd = torch.zeros(K, dtype=torch.float64, device="cuda")
        fgd.fgd_outer_step(fgd.Context(K, P), d2, fgd.MixDesc.mean(K), None, False, f_tl, f_tp, f_v, f_tp, 0.7, 0.9, cd)
        torch.cuda.synchronize()
        outs.append((f_tp.clone(), f_v.clone(), cd.clone()))
    assert all(torch.equal(a, b) for a, b in zip(*outs))


def test_argument_errors():
    K, P = 4, 1024
    ctx = fgd.Context(K, P)
    a = torch.zeros((K, P), device="cuda")
    b, c, d = torch.zeros_like(a), torch.zeros_like(a), torch.zeros_like(a)
    ring = fgd.MixDesc.ring(K)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_outer_grad(ctx, a, b, a)
    assert e.value.status == fgd.FGD_ERR_ALIAS
    with pytest.raises(fgd.FgdError) as e:   # momentum aliases theta_local
        fgd.fgd_outer_step(ctx, ring, fgd.MixDesc.mean(K), None, False, b, a, b, d)
    assert e.value.status == fgd.FGD_ERR_ALIAS
    with pytest.raises(fgd.FgdError) as e:   # partial overlap of theta_new and theta_prev
        big = torch.zeros(K * P + 8, device="cuda")
        fgd.fgd_outer_step(ctx, ring, fgd.MixDesc.mean(K), None, False, b, big[:K * P].view(K, P), c,
                           big[4:K * P + 4].view(K, P))
    assert e.value.status == fgd.FGD_ERR_ALIAS
    with pytest.raises(fgd.FgdError) as e:   # neither x nor mix1_fused
        fgd.fgd_outer_step(ctx, ring, None, None, False, b, a, c, d)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError) as e:   # descriptor for another K
        fgd.fgd_mix(ctx, fgd.MixDesc.ring(8), a, b)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG and "does not match" in e.value.message
    with pytest.raises(fgd.FgdError) as e:   # vector output only for the mean
        fgd.fgd_mix(ctx, ring, a, b[0], out_is_vector=True)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_outer_step(ctx, ring, fgd.MixDesc.dense(np.eye(K)), None, False, b, a, c, d)
    assert e.value.status == fgd.FGD_ERR_UNSUPPORTED
    with pytest.raises(fgd.FgdError):
        fgd.Context(4, 0)            # empty tensors are rejected, not launched
    with pytest.raises(fgd.FgdError):
        fgd.Context(0, 10)
    with pytest.raises(fgd.FgdError):
        fgd.Context(65, 10)
    with pytest.raises(fgd.FgdError):
        fgd.Context(4, 10, ld=8)
    # the context is still usable after errors
    fgd.fgd_outer_grad(ctx, a, b, c)
    torch.cuda.synchronize()


@pytest.mark.parametrize("K,P,mix1,mix2,rounds", [
    (8, 20000, ("mean",), ("matching", 0.05), 60),                          # the paper's setting, many rounds
    (64, 6000, ("ring", 0.1), ("dense", gen.sinkhorn_W(0, 64)), 30),        # tensor-core step and mix
    (48, 5000, ("mean",), ("ring",), 40),                                   # padded tensor-core shape
    (13, 30000, ("ring", 0.1), ("ring", 0.1), 30),                          # zero-padded onto the 16-worker fp32 kernel
])
def test_long_free_running_rounds(K, P, mix1, mix2, rounds):
    """Many free-running rounds (the oracle keeps its own float64 state): the fp32 path must not drift
    out of tolerance -- nothing accumulates beyond rounding, as a contraction with a doubly stochastic
    matrix cannot amplify it."""
    Scenario(K, P, mix1, mix2, seed=3, mode="factored").run(rounds)
