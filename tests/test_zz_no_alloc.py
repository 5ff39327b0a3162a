"""The allocation-free consensus-distance entry point (collected last on purpose).

It exists for callers that cannot allocate GPU memory (no context, no cudaMalloc): its partial
sums go through a fixed array inside the library.  The tests call it through the C ABI twice
in a row -- the second call finds the first call's leftovers in the shared array -- and check
both results against the context-based entry point and against the float64 oracle within the
consensus tolerance; they also check the property the entry point exists for (the device's free
memory does not move across calls), a launch on a stream other than the default one, and the
argument errors.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2606_22768_b200 as fgd
from fgd_inputs import gen

from tests.gpu_util import assert_cd_close

pytestmark = pytest.mark.gpu

CD_RTOL = 1e-5

# (K, P, ld): compile-time and run-time worker counts, a ragged row stride, a run-time K whose
# private columns need more than 48 KB of dynamic shared memory (63), and a compile-time K whose
# odd row stride forces the element-wise loads (16 with ld = P + 1)
SHAPES = [(16, 300001, 300004), (4, 1 << 20, 1 << 20), (5, 7777, 7780), (64, 20000, 20000),
          (63, 20011, 20012), (16, 40001, 40002), (8, 12345, 12345)]


def _padded(th, K, P, ld):
    full = torch.full((K, ld), -777.0, dtype=torch.float32, device="cuda")
    full[:, :P].copy_(torch.from_numpy(th))
    return full


@pytest.mark.parametrize("K,P,ld", SHAPES)
def test_noalloc_matches_context_entry_point_and_oracle_twice(K, P, ld):
    th_a = gen.theta0(21, K, P, 0.02, 7e-4)
    th_b = gen.theta0(22, K, P, 0.02, 2e-3)          # a second, different input: different sums
    ctx = fgd.Context(K, P, ld)
    for th in (th_a, th_b):
        full = _padded(th, K, P, ld)
        want = torch.zeros(K, dtype=torch.float64, device="cuda")
        got = torch.full((K,), -1.0, dtype=torch.float64, device="cuda")
        fgd.fgd_consensus_distance(ctx, full, want)
        fgd.fgd_consensus_distance_noalloc(0, K, P, ld, full, got)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert (w > 0).all()
        assert np.all(np.abs(g - w) <= CD_RTOL * np.abs(w)), f"noalloc {g} vs context {w}"
        assert_cd_close(g, oracle.consensus_sumsq(th.astype(np.float64)), P, "noalloc vs oracle")


def test_noalloc_leaves_free_memory_alone_and_runs_on_any_stream():
    K, P, ld = 16, 200003, 200004
    th = gen.theta0(23, K, P, 0.02, 1e-3)
    full = _padded(th, K, P, ld)
    got = torch.zeros((3, K), dtype=torch.float64, device="cuda")
    side = torch.cuda.Stream()
    fgd.fgd_consensus_distance_noalloc(0, K, P, ld, full, got[0])     # first call on the device: resolves the array
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    fgd.fgd_consensus_distance_noalloc(0, K, P, ld, full, got[1])     # current (default) stream
    torch.cuda.synchronize()                                          # calls share the array: keep them ordered
    fgd.fgd_consensus_distance_noalloc(0, K, P, ld, full, got[2], stream=side)
    side.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, f"device free memory moved by {free0 - free1} bytes across allocation-free calls"
    g = got.cpu().numpy()
    assert np.array_equal(g[0], g[1]) and np.array_equal(g[1], g[2])  # deterministic, whatever the stream
    assert_cd_close(g[2], oracle.consensus_sumsq(th.astype(np.float64)), P, "noalloc on a side stream vs oracle")


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    th = torch.zeros((4, 64), dtype=torch.float32, device="cuda")
    out = torch.zeros(80, dtype=torch.float64, device="cuda")
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_consensus_distance_noalloc(0, fgd.FGD_MAX_K + 1, 64, 64, th, out)
    assert e.value.status == fgd.FGD_ERR_INVALID_ARG and "static scratch" in e.value.message
    with pytest.raises(fgd.FgdError):
        fgd.fgd_consensus_distance_noalloc(0, 4, 64, 32, th, out)


def test_noalloc_rejects_an_output_inside_the_input():
    th = torch.zeros((4, 64), dtype=torch.float64, device="cuda")      # 4 x 128 floats when viewed as fp32
    as_f32 = th.view(torch.float32)
    with pytest.raises(fgd.FgdError) as e:
        fgd.fgd_consensus_distance_noalloc(0, 4, 128, 128, as_f32, th[1])
    assert e.value.status == fgd.FGD_ERR_ALIAS
