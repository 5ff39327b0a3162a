"""The whole round (side-stream Mix1, fused outer step, consensus finalisation) captured once into a
CUDA graph and replayed: same results as the eager calls, checked against the oracle every round."""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen
from paper_2606_22768_b200.round import OuterRound
from tests.gpu_util import assert_cd_close, assert_param_close, make_mix, upload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,P,mix1,mix2,fused", [
    (4, 1 << 16, ("mean",), ("ring",), False),            # the L2-resident latency configuration's structure
    (16, 50001, ("hypercube",), ("hypercube",), False),   # matrix-valued Mix1 result on the side stream
    (16, 30000, ("ring",), ("ring",), True),              # gossip Mix1 fused: one kernel + finalisation
    (64, 9000, ("mean",), ("dense", gen.sinkhorn_W(0, 64)), False),   # tensor-core kernel
    (40, 20001, ("ring",), ("matching",), True),          # row-gather step (gossip Mix1 fused, run-time worker count)
    (24, 7000, ("ring",), ("ring",), False),              # row-gather mix on the side stream + row-gather step with a matrix x
])
def test_round_replayed_from_a_cuda_graph(K, P, mix1, mix2, fused):
    seed = 5
    ld = P + (4 - P % 4) % 4
    th0 = gen.theta0(seed, K, P, 0.02, 5e-4)
    f_th, g_th = upload(th0, ld)
    f_v, g_v = upload(np.zeros((K, P), np.float32), ld)
    f_loc, g_loc = upload(th0, ld)
    d1, W1 = make_mix(mix1, K, 0, seed, 1)
    d2, W2 = make_mix(mix2, K, 0, seed, 2)
    drv = OuterRound(K, P, ld)

    def body():
        if fused:
            drv.step(d2, f_loc, f_th, f_v, f_th, 0.7, 0.9, mix1_fused=d1)
        else:
            drv.launch_mix1(d1, f_th)
            drv.step(d2, f_loc, f_th, f_v, f_th, 0.7, 0.9)

    o_th, o_v = th0.astype(np.float64), np.zeros((K, P))
    graph = None
    for r in range(4):
        drift = gen.scaled_normal(seed, gen.TENSOR_DRIFT, r, K, P, np.full(K, 1e-3, np.float32))
        g_loc.copy_(torch.from_numpy(g_th.cpu().numpy() + drift))
        if r == 0:
            body()                      # eager: sizes the launches, allocates the Mix1 buffers
            torch.cuda.synchronize()
            graph = drv.capture(body)   # capturing executes nothing
        else:
            graph.replay()
        torch.cuda.synchronize()
        o_th, o_v = oracle.outer_round(W1, W2, o_th, o_th + drift.astype(np.float64), o_v, 0.7, 0.9)
        assert_param_close(g_th, o_th, f"theta_new round {r}")
        assert_param_close(g_v, o_v, f"momentum round {r}")
        assert_cd_close(drv.cd_sumsq, oracle.consensus_sumsq(o_th), P, f"cd round {r}")
    fgd.fgd_device_status(drv.ctx)
