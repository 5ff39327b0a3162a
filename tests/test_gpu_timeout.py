"""A bounded device-side wait that runs out (no GPU is faulted, trapped or hung).

The pipelined kernels wait on shared-memory barriers with a poll limit.  The library's test hooks
shorten that limit and make every CTA's producer withhold the loads of one tile, so the consumers'
wait for that tile gives up: the kernel must record FGD_ERR_TIMEOUT in the context's status word,
wait for the copies it still has in flight, give its tensor memory back and return.  Checked for
the three kernel families that have such waits: fgd_device_status reports the timeout once, and
the same context then computes, bit for bit, what a fresh context computes.
"""
import numpy as np
import pytest
import torch

import paper_2606_22768_b200 as fgd
from fgd_inputs import gen

pytestmark = pytest.mark.gpu

SPIN = 4096          # polls before a wait gives up in the shortened runs


def _inputs(K, P, seed):
    th = torch.from_numpy(gen.theta0(seed, K, P, 0.02, 5e-4)).cuda()
    loc = th + torch.from_numpy(gen.scaled_normal(seed, gen.TENSOR_DRIFT, 0, K, P, np.full(K, 1e-3, np.float32))).cuda()
    mom = torch.from_numpy(gen.scaled_normal(seed, gen.TENSOR_MOMENTUM, 0, K, P, 1e-3)).cuda()
    return th, loc, mom


def _step(ctx, m2, th, loc, mom, x):
    cd = torch.zeros(ctx.K, dtype=torch.float64, device="cuda")
    fgd.fgd_outer_step(ctx, m2, None, x, True, loc, th, mom, th, 0.7, 0.9, cd)
    return cd


def _expect_timeout_once(ctx):
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_device_status(ctx)
    assert e.value.status == fgd.FGD_ERR_TIMEOUT
    fgd.fgd_device_status(ctx)          # the flag was cleared: no second report


@pytest.mark.parametrize("K,P,mix2", [(4, 148 * 4 * 1024 + 52, "ring"),      # fp32 TMA pipeline, four tiles per CTA
                                      (64, 148 * 4 * 128 + 36, "dense")])    # tcgen05 step
def test_fused_step_wait_runs_out_and_context_recovers(K, P, mix2):
    m2 = fgd.MixDesc.ring(K) if mix2 == "ring" else fgd.MixDesc.dense(gen.sinkhorn_W(3, K))
    th0, loc0, mom0 = _inputs(K, P, 31)
    x = th0.mean(0).contiguous()
    ctx = fgd.Context(K, P)
    fgd.fgd_set_path(ctx, fgd.FGD_PATH_TMA)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, SPIN)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, 1)
    th, mom = th0.clone(), mom0.clone()
    _step(ctx, m2, th, loc0, mom, x)                       # returns: the launch is asynchronous
    _expect_timeout_once(ctx)
    # hooks off: the same context must now behave like a new one
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, 0)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, -1)
    th, mom = th0.clone(), mom0.clone()
    cd = _step(ctx, m2, th, loc0, mom, x)
    fgd.fgd_device_status(ctx)
    fresh = fgd.Context(K, P)
    fgd.fgd_set_path(fresh, fgd.FGD_PATH_TMA)
    th_f, mom_f = th0.clone(), mom0.clone()
    cd_f = _step(fresh, m2, th_f, loc0, mom_f, x)
    fgd.fgd_device_status(fresh)
    assert torch.equal(th, th_f) and torch.equal(mom, mom_f) and torch.equal(cd, cd_f)
    assert not torch.equal(th, th0)                        # and it did compute something


def test_gossip_tensor_core_step_wait_runs_out_and_context_recovers():
    """The step with a sparse Mix1 fused (both mixes as MMAs, ring of single boxes)."""
    K, P = 64, 148 * 4 * 128 + 36
    m1, m2 = fgd.MixDesc.hypercube(K), fgd.MixDesc.ring(K)   # six neighbour slots: Mix1 runs as MMAs
    th0, loc0, mom0 = _inputs(K, P, 33)

    def run(ctx, th, mom):
        cd = torch.zeros(K, dtype=torch.float64, device="cuda")
        fgd.fgd_outer_step(ctx, m2, m1, None, False, loc0, th, mom, th, 0.7, 0.9, cd)
        return cd

    _gossip_timeout_case(K, P, run, th0, mom0, gossip_path=2)


def test_row_gather_step_wait_runs_out_and_context_recovers():
    """The step with a sparse Mix1 fused above 32 workers (TMA-pipelined row gather, run-time worker count)."""
    K, P = 40, 148 * 4 * 128 + 36
    m1, m2 = fgd.MixDesc.ring(K), fgd.MixDesc.ring(K)
    th0, loc0, mom0 = _inputs(K, P, 35)

    def run(ctx, th, mom):
        cd = torch.zeros(K, dtype=torch.float64, device="cuda")
        fgd.fgd_outer_step(ctx, m2, m1, None, False, loc0, th, mom, th, 0.7, 0.9, cd)
        return cd

    _gossip_timeout_case(K, P, run, th0, mom0, gossip_path=3)


def _gossip_timeout_case(K, P, run, th0, mom0, gossip_path):
    ctx = fgd.Context(K, P)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_GOSSIP_PATH, gossip_path)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, SPIN)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, 1)
    run(ctx, th0.clone(), mom0.clone())
    _expect_timeout_once(ctx)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, 0)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, -1)
    th, mom = th0.clone(), mom0.clone()
    cd = run(ctx, th, mom)
    fgd.fgd_device_status(ctx)
    fresh = fgd.Context(K, P)
    fgd.fgd_debug_set(fresh, fgd.FGD_DEBUG_GOSSIP_PATH, gossip_path)
    th_f, mom_f = th0.clone(), mom0.clone()
    cd_f = run(fresh, th_f, mom_f)
    fgd.fgd_device_status(fresh)
    assert torch.equal(th, th_f) and torch.equal(mom, mom_f) and torch.equal(cd, cd_f)
    assert not torch.equal(th, th0)


def test_tensor_core_mix_wait_runs_out_and_context_recovers():
    K, P = 64, 148 * 4 * 128 + 36
    W = fgd.MixDesc.dense(gen.sinkhorn_W(5, K))
    th0, _, _ = _inputs(K, P, 32)
    ctx = fgd.Context(K, P)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, SPIN)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, 2)
    out = torch.zeros_like(th0)
    fgd.fgd_mix(ctx, W, th0, out)
    _expect_timeout_once(ctx)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, 0)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, -1)
    out.zero_()
    fgd.fgd_mix(ctx, W, th0, out)
    fgd.fgd_device_status(ctx)
    fresh, out_f = fgd.Context(K, P), torch.zeros_like(th0)
    fgd.fgd_mix(fresh, W, th0, out_f)
    fgd.fgd_device_status(fresh)
    assert torch.equal(out, out_f) and bool((out != 0).any())


def test_gather_mix_wait_runs_out_and_context_recovers():
    """The stand-alone sparse mix above 16 workers (TMA-pipelined row gather, run-time worker count)."""
    K, P = 40, 148 * 4 * 4 * 128 + 36          # more tiles than stages for every CTA at four CTAs per SM
    W = fgd.MixDesc.ring(K)
    th0, _, _ = _inputs(K, P, 34)
    ctx = fgd.Context(K, P)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, SPIN)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, 2)
    out = torch.zeros_like(th0)
    fgd.fgd_mix(ctx, W, th0, out)
    _expect_timeout_once(ctx)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SPIN_LIMIT, 0)
    fgd.fgd_debug_set(ctx, fgd.FGD_DEBUG_SKIP_TILE, -1)
    out.zero_()
    fgd.fgd_mix(ctx, W, th0, out)
    fgd.fgd_device_status(ctx)
    fresh, out_f = fgd.Context(K, P), torch.zeros_like(th0)
    fgd.fgd_mix(fresh, W, th0, out_f)
    fgd.fgd_device_status(fresh)
    assert torch.equal(out, out_f) and bool((out != 0).any())


def test_debug_set_rejects_unknown_keys():
    ctx = fgd.Context(4, 1024)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_debug_set(ctx, 99, 1)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG
