"""The access-pattern probe (fgd_debug_stream_pattern): it must move data without changing it."""
import numpy as np
import pytest
import torch

import paper_2606_22768_b200 as fgd
from fgd_inputs import gen

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,P,ld", [(64, 148 * 3 * 128 + 77, 148 * 3 * 128 + 80), (16, 200003, 200004), (8, 70000, 70000),
                                    (4, 5000, 5000), (32, 40001, 40004)])
def test_probe_copies_theta_prev_and_keeps_the_momentum(K, P, ld):
    th = torch.full((K, ld), -777.0, device="cuda")
    th[:, :P] = torch.from_numpy(gen.theta0(41, K, P, 0.02, 1e-3)).cuda()
    loc = th + 1e-3
    mom = torch.full((K, ld), -777.0, device="cuda")
    mom[:, :P] = torch.from_numpy(gen.scaled_normal(41, gen.TENSOR_MOMENTUM, 0, K, P, 1e-3)).cuda()
    th0, mom0 = th.clone(), mom.clone()
    ctx = fgd.Context(K, P, ld)
    out = torch.full((K, ld), -777.0, device="cuda")
    fgd.fgd_debug_stream_pattern(ctx, loc, th, mom, out)           # out of place
    fgd.fgd_debug_stream_pattern(ctx, loc, th, mom, th)            # in place
    fgd.fgd_device_status(ctx)
    assert torch.equal(out, th0) and torch.equal(th, th0) and torch.equal(mom, mom0)   # padding columns included


def test_probe_argument_errors():
    ctx = fgd.Context(5, 1024)
    t = torch.zeros((5, 1024), device="cuda")
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_debug_stream_pattern(ctx, t.clone(), t, t.clone(), t)
    assert e.value.status == fgd.FGD_ERR_UNSUPPORTED
    ctx = fgd.Context(8, 1024)
    t = torch.zeros((8, 1024), device="cuda")
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_debug_stream_pattern(ctx, t, t, t.clone(), t)      # theta_local aliases theta_new
    assert e.value.status == fgd.FGD_ERR_ALIAS
