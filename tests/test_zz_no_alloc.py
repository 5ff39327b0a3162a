"""The allocation-free consensus-distance entry point (collected last on purpose).

It exists for callers that cannot allocate GPU memory (no context, no cudaMalloc): its partial
sums go through a fixed array inside the library.  The test calls it through the C ABI twice
in a row -- the second call finds the first call's leftovers in the shared array -- and checks
both results against the context-based entry point within the consensus tolerance.
"""
import numpy as np
import pytest
import torch

import paper_2606_22768_b200 as fgd
from fgd_inputs import gen

pytestmark = pytest.mark.gpu

CD_RTOL = 1e-5


@pytest.mark.parametrize("K,P,ld", [(16, 300001, 300004), (4, 1 << 20, 1 << 20), (5, 7777, 7780), (64, 20000, 20000)])
def test_noalloc_matches_context_entry_point_twice(K, P, ld):
    th_a = gen.theta0(21, K, P, 0.02, 7e-4)
    th_b = gen.theta0(22, K, P, 0.02, 2e-3)          # a second, different input: different sums
    ctx = fgd.Context(K, P, ld)
    for th in (th_a, th_b):
        full = torch.full((K, ld), -777.0, dtype=torch.float32, device="cuda")
        full[:, :P].copy_(torch.from_numpy(th))
        want = torch.zeros(K, dtype=torch.float64, device="cuda")
        got = torch.full((K,), -1.0, dtype=torch.float64, device="cuda")
        fgd.fgd_consensus_distance(ctx, full, want)
        fgd.fgd_consensus_distance_noalloc(0, K, P, ld, full, got)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert (w > 0).all()
        assert np.all(np.abs(g - w) <= CD_RTOL * np.abs(w)), f"noalloc {g} vs context {w}"


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    th = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    out = torch.zeros(80, dtype=torch.float64, device="cuda")
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_consensus_distance_noalloc(0, fgd.FGD_MAX_K + 1, 64, 64, th, out)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG and "static scratch" in e.value.message
    with pytest.raises(fgd.FgdError):
        fgd.fgd_consensus_distance_noalloc(0, 4, 64, 32, th, out)
