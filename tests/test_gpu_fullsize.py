"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

The [K, P] tensors are generated in HBM by the seeded generator's CUDA twin; because every value
is a pure function of (seed, tensor, round, worker, column), the oracle regenerates any column
block on the CPU and runs the SAME multi-round recursion on it (columns are independent), free
running in float64.  Compared per round on sampled column blocks (first, last with the ragged
tail, blocks straddling tile boundaries): theta_new and momentum element-wise.  Over ALL columns:
the fused consensus sums of the last round against the oracle's (every configuration), and as
properties -- every round the fused sums equal the stand-alone kernel's, a stand-alone call on a
sampled window equals the oracle on that window, and round 0 lands on the closed-form
expectation of the consensus distance.
"""
import os
import sys

import numpy as np
import pytest
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen, gpu as inputs_gpu
from paper_2606_22768_b200.round import OuterRound
from tests.gpu_util import assert_cd_close, assert_param_close, make_mix

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402  (the configs and mix schedule the benchmark uses)

pytestmark = pytest.mark.gpu

WIDTH = 1536


def _blocks(P, rng):
    starts = [0, P - WIDTH, 509, (P // 2) - 3]
    starts += [int(x) for x in rng.integers(WIDTH, P - 2 * WIDTH, 4)]
    return sorted(set(max(0, min(P - WIDTH, s)) for s in starts))


def _spec(cfg, which):
    kind = cfg[which][0]
    if kind == "dense":
        return ("dense", gen.sinkhorn_W(0, cfg["K"]))
    if cfg["p_fail"] > 0 and kind in ("ring", "xor", "hypercube", "matching"):
        return (kind, cfg["p_fail"], fgd.FGD_RENORM_METROPOLIS)
    return (kind,)


@pytest.mark.parametrize("cfg_id,rounds", [(2, 10), (3, 10), (4, 20), (5, 5), (6, 3)])
def test_full_size_config(cfg_id, rounds):
    cfg = bench.CONFIGS[cfg_id]
    K, P, seed = cfg["K"], cfg["P"], 0
    need = (4 if cfg["mix1"][0] != "mean" else 3) * K * P * 4 + 4 * P + (2 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free HBM for this configuration")
    sig = (gen.drift_sigmas(seed, K, *cfg["sig"]) if cfg["sig"][0] != cfg["sig"][1]
           else np.full(K, cfg["sig"][0], np.float32))
    theta = torch.empty((K, P), dtype=torch.float32, device="cuda")
    local = torch.empty_like(theta)
    mom = torch.zeros_like(theta)
    inputs_gpu.theta0(theta, seed)
    drv = OuterRound(K, P)
    cd_alone = torch.zeros(K, dtype=torch.float64, device="cuda")
    rng = np.random.default_rng(cfg_id)
    blocks = _blocks(P, rng)
    o_theta = {p0: gen.theta0(seed, K, P, p0=p0, p1=p0 + WIDTH).astype(np.float64) for p0 in blocks}
    o_v = {p0: np.zeros((K, WIDTH)) for p0 in blocks}
    s1, s2 = _spec(cfg, "mix1"), _spec(cfg, "mix2")

    for r in range(rounds):
        d1, W1 = make_mix(s1, K, r, seed, 1)
        d2, W2 = make_mix(s2, K, r, seed, 2)
        drv.launch_mix1(d1, theta)                                # side stream
        inputs_gpu.local_steps(local, theta, sig, seed, r)        # stand-in for the inner steps
        drv.step(d2, local, theta, mom, theta, 0.7, 0.9)          # in place, fused consensus sums
        fgd.fgd_consensus_distance(drv.ctx, theta, cd_alone)
        torch.cuda.synchronize()
        # all columns: two different kernels must agree on the consensus sums
        fused = drv.cd_sumsq.cpu().numpy()
        alone = cd_alone.cpu().numpy()
        assert np.all(np.abs(fused - alone) <= 2e-6 * np.abs(alone)), f"round {r}: fused {fused} vs stand-alone {alone}"
        if r == 0 and cfg_id in (2, 3):
            # closed form for Mix1 = mean, v = 0, iid drift: E[CD_sq] = P g^2 (1+mu)^2 mean(sigma^2) (|W2|_F^2 - 1)/K
            expect = P * 0.7 ** 2 * 1.9 ** 2 * float(np.mean(sig.astype(np.float64) ** 2)) * ((W2 * W2).sum() - 1.0) / K
            assert fgd.fgd_cd_finalize(fused)[1] == pytest.approx(expect, rel=2e-3)
        # sampled blocks: free-running float64 oracle on regenerated inputs
        for p0 in blocks:
            drift = gen.scaled_normal(seed, gen.TENSOR_DRIFT, r, K, P, sig, p0, p0 + WIDTH).astype(np.float64)
            o_theta[p0], o_v[p0] = oracle.outer_round(W1, W2, o_theta[p0], o_theta[p0] + drift, o_v[p0], 0.7, 0.9)
            assert_param_close(theta[:, p0:p0 + WIDTH], o_theta[p0], f"cfg{cfg_id} round {r} theta_new block {p0}")
            assert_param_close(mom[:, p0:p0 + WIDTH], o_v[p0], f"cfg{cfg_id} round {r} momentum block {p0}")
    fgd.fgd_device_status(drv.ctx)
    # the fused consensus sums of the last round against the oracle over ALL columns, at the launch
    # shape the benchmark times (columns are independent, so the oracle takes them in chunks of
    # 2^28 / K columns and the per-worker sums add up)
    total = np.zeros(K)
    chunk = (1 << 28) // K
    for c0 in range(0, P, chunk):
        total += oracle.consensus_sumsq(theta[:, c0:min(P, c0 + chunk)].cpu().numpy())
    assert_cd_close(drv.cd_sumsq, total, P, f"cfg{cfg_id} fused consensus sums, all columns")
    # a stand-alone consensus call on a sampled window (row stride P, 16-byte aligned start)
    p0 = blocks[len(blocks) // 2] // 4 * 4
    win = fgd.Context(K, WIDTH, P)
    out = torch.zeros(K, dtype=torch.float64, device="cuda")
    fgd.fgd_consensus_distance(win, theta[:, p0:], out)
    torch.cuda.synchronize()
    ref = oracle.consensus_sumsq(theta[:, p0:p0 + WIDTH].cpu().numpy())
    assert_cd_close(out, ref, WIDTH, "window consensus")
    del theta, local, mom
    torch.cuda.empty_cache()


def test_more_than_2_to_31_columns():
    """Maximum sizes: P just above 2^31 columns (64-bit column arithmetic end to end; the TMA kernels'
    32-bit box coordinates do not reach that far, so AUTO must pick the register kernels and a forced
    TMA path must refuse).  K = 3 ring, 2 rounds, sampled blocks around 0, 2^31 and the ragged end."""
    K, P, seed = 3, (1 << 31) + 4102, 11
    need = 3 * K * P * 4 + P * 4 + (2 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free HBM for this size")
    sig = np.full(K, 1e-3, np.float32)
    theta = torch.empty((K, P), dtype=torch.float32, device="cuda")
    local = torch.empty_like(theta)
    mom = torch.zeros_like(theta)
    inputs_gpu.theta0(theta, seed)
    drv = OuterRound(K, P)
    blocks = [0, (1 << 31) - 700, (1 << 31) + 2000, P - WIDTH, (1 << 30) + 12345]
    o_theta = {p0: gen.theta0(seed, K, P, p0=p0, p1=p0 + WIDTH).astype(np.float64) for p0 in blocks}
    o_v = {p0: np.zeros((K, WIDTH)) for p0 in blocks}
    cd_alone = torch.zeros(K, dtype=torch.float64, device="cuda")
    for r in range(2):
        d1, W1 = make_mix(("mean",), K, r, seed, 1)
        d2, W2 = make_mix(("ring", 0.2), K, r, seed, 2)
        drv.launch_mix1(d1, theta)
        inputs_gpu.local_steps(local, theta, sig, seed, r)
        drv.step(d2, local, theta, mom, theta, 0.7, 0.9)
        fgd.fgd_consensus_distance(drv.ctx, theta, cd_alone)
        torch.cuda.synchronize()
        fused, alone = drv.cd_sumsq.cpu().numpy(), cd_alone.cpu().numpy()
        assert np.all(np.abs(fused - alone) <= 2e-6 * np.abs(alone)), f"round {r}: fused {fused} vs stand-alone {alone}"
        for p0 in blocks:
            drift = gen.scaled_normal(seed, gen.TENSOR_DRIFT, r, K, P, sig, p0, p0 + WIDTH).astype(np.float64)
            o_theta[p0], o_v[p0] = oracle.outer_round(W1, W2, o_theta[p0], o_theta[p0] + drift, o_v[p0], 0.7, 0.9)
            assert_param_close(theta[:, p0:p0 + WIDTH], o_theta[p0], f"round {r} theta_new block {p0}")
            assert_param_close(mom[:, p0:p0 + WIDTH], o_v[p0], f"round {r} momentum block {p0}")
    fgd.fgd_device_status(drv.ctx)
    fgd.fgd_set_path(drv.ctx, fgd.FGD_PATH_TMA)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_outer_step(drv.ctx, d2, d1, None, False, local, theta, mom, theta, 0.7, 0.9, None)
    assert e.value.status == fgd.FGD_ERR_UNSUPPORTED
    del theta, local, mom
    torch.cuda.empty_cache()


@pytest.mark.parametrize("K,P,mix1,fused", [(40, 40_000_037, ("mean",), False),      # padded to 48 workers, ragged tail
                                            (56, 30_000_004, ("ring", 0.1), True),   # row gather, gossip Mix1 fused (56 rows, nothing padded)
                                            (12, 100_000_002, ("ring",), False),     # compile-time 12, matrix-valued x
                                            (13, 70_000_004, ("mean",), False),      # zero-padded onto the 16-worker fp32 kernel
                                            (10, 50_000_002, ("ring", 0.1), True),   # zero-padded onto 12, gossip Mix1 fused
                                            (64, 20_000_003, ("ring", 0.1), True),   # row gather with the gossip Mix1 fused, ragged tail
                                            (64, 20_000_003, ("hypercube", 0.1), True),   # both mixes as MMAs, ragged tail
                                            (24, 60_000_002, ("ring", 0.1), False),       # row gather, matrix-valued x, two CTAs per SM, ragged tail
                                            (48, 30_000_001, ("matching", 0.1), False)])  # row gather, matrix-valued x, one CTA per SM
def test_full_size_other_worker_counts(K, P, mix1, fused):
    """Worker counts beside the benchmark configurations at sizes of many thousand tiles per CTA:
    zero-padded tensor-core shapes and the 12-worker kernel, 3 free-running rounds, sampled blocks."""
    seed = 21
    ld = (P + 3) // 4 * 4
    need = 4 * K * ld * 4 + (2 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free HBM for this size")
    sig = np.full(K, 1e-3, np.float32)
    full = [torch.full((K, ld), -777.0, dtype=torch.float32, device="cuda") for _ in range(3)]
    theta, local, mom = (t[:, :P] for t in full)
    inputs_gpu.theta0(theta, seed)
    mom.zero_()
    drv = OuterRound(K, P, ld)
    blocks = sorted({0, P - WIDTH, 127 * 1000 + 5, (P // 2) // 128 * 128 - 40, P // 3})
    o_theta = {p0: gen.theta0(seed, K, P, p0=p0, p1=p0 + WIDTH).astype(np.float64) for p0 in blocks}
    o_v = {p0: np.zeros((K, WIDTH)) for p0 in blocks}
    cd_alone = torch.zeros(K, dtype=torch.float64, device="cuda")
    for r in range(3):
        d1, W1 = make_mix(mix1, K, r, seed, 1)
        d2, W2 = make_mix(("ring", 0.2), K, r, seed, 2)
        inputs_gpu.local_steps(local, theta, sig, seed, r)
        if fused:
            drv.step(d2, full[1], full[0], full[2], full[0], 0.7, 0.9, mix1_fused=d1)
        else:
            drv.launch_mix1(d1, full[0])
            drv.step(d2, full[1], full[0], full[2], full[0], 0.7, 0.9)
        fgd.fgd_consensus_distance(drv.ctx, full[0], cd_alone)
        torch.cuda.synchronize()
        fused_cd, alone = drv.cd_sumsq.cpu().numpy(), cd_alone.cpu().numpy()
        assert np.all(np.abs(fused_cd - alone) <= 2e-6 * np.abs(alone)), f"round {r}: fused {fused_cd} vs stand-alone {alone}"
        for p0 in blocks:
            drift = gen.scaled_normal(seed, gen.TENSOR_DRIFT, r, K, P, sig, p0, p0 + WIDTH).astype(np.float64)
            o_theta[p0], o_v[p0] = oracle.outer_round(W1, W2, o_theta[p0], o_theta[p0] + drift, o_v[p0], 0.7, 0.9)
            assert_param_close(theta[:, p0:p0 + WIDTH], o_theta[p0], f"K={K} round {r} theta_new block {p0}")
            assert_param_close(mom[:, p0:p0 + WIDTH], o_v[p0], f"K={K} round {r} momentum block {p0}")
    fgd.fgd_device_status(drv.ctx)
    for t in full:
        if ld > P:
            assert bool((t[:, P:] == -777.0).all()), "padding columns were written"
    del theta, local, mom, full
    torch.cuda.empty_cache()
