// Host side of the TMA-pipelined fused outer step: eligibility, tensor maps, kernel selection.
#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_mix_dense_tc.cuh"
#include "fgd_step_dense_tc.cuh"
#include "fgd_step_gossip_tc.cuh"
#include "fgd_tma_host.h"

using namespace fgd;

int fgd_launch_step_tma_g0(fgd_ctx*, const StepArgs&, bool, const GatherMix&, const DenseMix&, const GatherMix&, FgdTmaShape, cudaStream_t, int*);
int fgd_launch_step_tma_g1(fgd_ctx*, const StepArgs&, bool, const GatherMix&, const DenseMix&, const GatherMix&, FgdTmaShape, cudaStream_t, int*);
int fgd_launch_step_tma_g2(fgd_ctx*, const StepArgs&, bool, const GatherMix&, const DenseMix&, const GatherMix&, FgdTmaShape, cudaStream_t, int*);
int fgd_launch_step_tma_g3(fgd_ctx*, const StepArgs&, bool, const GatherMix&, const DenseMix&, const GatherMix&, FgdTmaShape, cudaStream_t, int*);

// Tensor-core dense step: Mix1 given (row or matrix) or fused (mean or gossip); K = 64 and every worker
// count in [17, 63] that has no compile-time fp32 kernel of its own (zero-padded to 32, 48 or 64),
// plus K = 32 when the caller says so (`tc_at_32`: a dense Mix2, or a sparse one the fp32 kernel
// is slow on).
bool fgd_tc_eligible(const fgd_ctx* c, const StepArgs& a, bool tc_at_32, const GatherMix& g1) {
  const int K = c->K;
  if (K > kTcMaxK || K < kTcMinK) return false;
  if (kt_of(K) == 16 || (kt_of(K) == 32 && !tc_at_32)) return false;
  if (!c->encode_tiled) return false;
  // column-range Mix2 is built for the one-value-per-column Mix1 (the "-subset" configurations pair it
  // with the global average)
  if (a.n_ranges != 0 && !(a.xsrc == XSRC_VECTOR || (a.xsrc == XSRC_FUSED && g1.kind == KMIX_MEAN))) return false;
  if (c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  return (size_t)c->max_smem_optin >= TcShape<kTcMaxK>::kSmem + 2304;   // + static shared memory (barriers, exchange rows)
}

template <int KP>
static int launch_tc(fgd_ctx* c, const TmaStepArgs& ta, const DenseMix& d2, const GatherMix& g1, cudaStream_t st, int* grid) {
  using Shape = TcShape<KP>;
  const StepArgs& a = ta.s;
  CUtensorMap tp, tl, tm, tx;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, kTcCols, KP)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, kTcCols, KP)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, kTcCols, KP)) return rc;
  tx = tp;                                    // n_tensors == 4: x has a map of its own (L2 prefetch only)
  if (ta.n_tensors == 4)
    if (int rc = make_tensor_map(c, &tx, a.x, kTcCols, KP)) return rc;
  const int64_t ntiles = (c->P + kTcCols - 1) / kTcCols;
  auto launch = [&](auto kern, int groups = 1) -> int {
    const int block = groups * kTcConsumers + 32;
    if (int r = persistent_grid(c, kern, block, Shape::kSmem, ntiles, grid)) return r;
    kern<<<*grid, block, Shape::kSmem, st>>>(ta, d2, g1, tp, tl, tm, tx);
    return FGD_OK;
  };
  const bool full = c->K == KP;
  const int xm = a.xsrc == XSRC_MATRIX ? 1 : ((a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER) ? 2 : 0);
  switch (xm) {
    case 1: return full ? launch(outer_step_dense_tc_kernel<KP, 1, true>) : launch(outer_step_dense_tc_kernel<KP, 1, false>);
    case 2:
      // A sparse Mix1 fused.  The gather from the stage costs one shared-memory load and one FMA per
      // neighbour slot and row (indices and weights are immediate constant-bank operands); running Mix1
      // as a second MMA group with the operands in tensor memory (fgd_step_gossip_tc.cuh) costs the
      // same whatever the slot count.  Measured at K = 64, same mix on both sides, TB/s gather / MMAs:
      // matching 5.24 / 4.69, ring 5.32 / 5.06, four slots 4.55 / 4.68, six (hypercube) 3.72 / 4.70 --
      // so three slots and more take the MMAs.  At the 32- and 48-worker shapes the per-tile latencies
      // of the MMA chain weigh more (K = 32: 4.0 TB/s against 4.7 for the gather at five slots).
      if constexpr (KP == 64) {
        // one or two neighbour slots: the gather is cheaper than the second MMA group
        if (c->dbg_gossip_path == 1 || (c->dbg_gossip_path == 0 && g1.D <= 2))
          return full ? launch(outer_step_dense_tc_kernel<KP, 2, true>) : launch(outer_step_dense_tc_kernel<KP, 2, false>);
        auto launch_g = [&](auto kern) -> int {
          const int block = TcGossipShape<KP>::kThreads;
          if (int r = persistent_grid(c, kern, block, TcGossipShape<KP>::kSmem, ntiles, grid)) return r;
          kern<<<*grid, block, TcGossipShape<KP>::kSmem, st>>>(ta, d2, g1, tp, tl, tm);
          return FGD_OK;
        };
        return full ? launch_g(outer_step_gossip_tc_kernel<KP, true>) : launch_g(outer_step_gossip_tc_kernel<KP, false>);
      } else if constexpr (KP == 32) {   // two consumer groups where the registers allow it
        return full ? launch(outer_step_dense_tc_kernel<KP, 2, true, false, 2>, 2) : launch(outer_step_dense_tc_kernel<KP, 2, false, false, 2>, 2);
      } else {
        return full ? launch(outer_step_dense_tc_kernel<KP, 2, true>) : launch(outer_step_dense_tc_kernel<KP, 2, false>);
      }
    default:
      if (a.n_ranges != 0)
        return full ? launch(outer_step_dense_tc_kernel<KP, 0, true, true>) : launch(outer_step_dense_tc_kernel<KP, 0, false, true>);
      if constexpr (KP == 32)      // two consumer groups where the registers allow it
        return full ? launch(outer_step_dense_tc_kernel<KP, 0, true, false, 2>, 2) : launch(outer_step_dense_tc_kernel<KP, 0, false, false, 2>, 2);
      else
        return full ? launch(outer_step_dense_tc_kernel<KP, 0, true>) : launch(outer_step_dense_tc_kernel<KP, 0, false>);
  }
}

int fgd_launch_step_dense_tc(fgd_ctx* c, const StepArgs& a, const DenseMix& d2, const GatherMix& g1, cudaStream_t st,
                             int* grid_out) {
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = (a.xsrc == XSRC_MATRIX && aligned16(a.x)) ? 4 : 3;
  ta.spin_limit = c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit;
  ta.skip_tile = c->dbg_skip_tile;
  int rc = FGD_OK;
  switch (tc_padded_k(c->K)) {
    case 32: ta.stages = TcShape<32>::kStages; rc = launch_tc<32>(c, ta, d2, g1, st, grid_out); break;
    case 48: ta.stages = TcShape<48>::kStages; rc = launch_tc<48>(c, ta, d2, g1, st, grid_out); break;
    default: ta.stages = TcShape<64>::kStages; rc = launch_tc<64>(c, ta, d2, g1, st, grid_out); break;
  }
  if (rc) return rc;
  return check_launch(c, "outer_step_dense_tc_kernel");
}

// Stand-alone mix on the tensor cores: same worker counts as the step (K = 32 only for a really
// dense matrix: its sparse fp32 kernel is at the copy roofline already).
bool fgd_mix_tc_eligible(const fgd_ctx* c, const float* in, bool really_dense) {
  const int K = c->K;
  if (K > kTcMaxK || K < kTcMinK || kt_of(K) == 16 || (kt_of(K) == 32 && !really_dense)) return false;
  if (!c->encode_tiled || c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096 || !aligned16(in)) return false;
  return (size_t)c->max_smem_optin >= TcMixShape<kTcMaxK>::kSmem + 512;
}

template <int KP>
static int launch_mix_tc(fgd_ctx* c, const TcMixArgs& a, const DenseMix& dm, cudaStream_t st) {
  CUtensorMap tin;
  if (int rc = make_tensor_map(c, &tin, a.in, kTcCols, KP)) return rc;
  const int64_t ntiles = (c->P + kTcCols - 1) / kTcCols;
  int grid = 0;
  auto launch = [&](auto kern) -> int {
    if (int r = persistent_grid(c, kern, TcMixShape<KP>::kThreads, TcMixShape<KP>::kSmem, ntiles, &grid)) return r;
    kern<<<grid, TcMixShape<KP>::kThreads, TcMixShape<KP>::kSmem, st>>>(a, dm, tin);
    return FGD_OK;
  };
  return c->K == KP ? launch(mix_dense_tc_kernel<KP, true>) : launch(mix_dense_tc_kernel<KP, false>);
}

int fgd_launch_mix_dense_tc(fgd_ctx* c, const float* in, float* out, const DenseMix& dm, cudaStream_t st) {
  const TcMixArgs a{in, out, c->P, c->ld, c->K, c->status, c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit, c->dbg_skip_tile};
  int rc = FGD_OK;
  switch (tc_padded_k(c->K)) {
    case 32: rc = launch_mix_tc<32>(c, a, dm, st); break;
    case 48: rc = launch_mix_tc<48>(c, a, dm, st); break;
    default: rc = launch_mix_tc<64>(c, a, dm, st); break;
  }
  if (rc) return rc;
  return check_launch(c, "mix_dense_tc_kernel");
}

bool fgd_tma_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, bool heavy, FgdTmaShape* out) {
  TmaShape sh{0, 0, 0};
  // `heavy` asks for the 512-consumer shape; worker counts without one fall back to the usual shapes
  if (!(heavy && tma_eligible(c, a, dense2, true, &sh)) && !tma_eligible(c, a, dense2, false, &sh)) return false;
  out->vec = sh.vec;
  out->consumers = sh.consumers;
  out->stages = sh.stages;
  return true;
}

int fgd_launch_step_tma(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                        const GatherMix& g1, FgdTmaShape shape, cudaStream_t st, int* grid_out) {
  switch (kt_tma_of(c->K)) {
    case 3: case 6: case 12: return fgd_launch_step_tma_g3(c, a, dense2, g2, d2, g1, shape, st, grid_out);
    case 0: case 2: case 4: return fgd_launch_step_tma_g0(c, a, dense2, g2, d2, g1, shape, st, grid_out);
    case 8: case 32: return fgd_launch_step_tma_g1(c, a, dense2, g2, d2, g1, shape, st, grid_out);
    default: return fgd_launch_step_tma_g2(c, a, dense2, g2, d2, g1, shape, st, grid_out);
  }
}
