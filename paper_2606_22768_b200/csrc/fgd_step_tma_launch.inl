// Kernel selection and launch of the TMA-pipelined fused step for ONE group of worker counts
// (FGD_TMA_GROUP); the groups are separate translation units so that they compile in parallel.
#include "fgd_tma_host.h"

using namespace fgd;

namespace {
static int launch_step_tma_group(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                    const GatherMix& g1, TmaShape sh, cudaStream_t st, int* grid_out) {
  const int KT = kt_tma_of(c->K), K = KT > 0 ? KT : c->K;      // K: rows of a tile; KT > c->K: zero-padded worker count
  const bool pad = KT > 0 && KT != c->K;
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = tma_n_tensors(a, KT, dense2);
  ta.stages = sh.stages;
  ta.spin_limit = c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit;
  ta.skip_tile = c->dbg_skip_tile;
  const int T = sh.consumers * sh.vec;
  const int boxc = T < 256 ? T : 256;
  CUtensorMap tp, tl, tm, tx;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, boxc, K)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, boxc, K)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, boxc, K)) return rc;
  if (int rc = make_tensor_map(c, &tx, a.xsrc == XSRC_MATRIX ? a.x : a.theta_prev, boxc, K)) return rc;
  const size_t smem = tma_fixed_smem(K, KT, dense2, sh.consumers) + tma_stage_bytes(K, T, ta.n_tensors) * sh.stages;
  const int64_t ntiles = (c->P + T - 1) / T;
  // neighbour count of a gather Mix2 as a template argument when it is one of the common ones
  // (identity 0, one-peer / matching 1, ring 2, hypercube of 16 workers 4); else read at run time
  int d2t = -1;
  // (three slots run as four, five to seven as eight: unused slots carry weight 0 and point at the
  // row itself; the eight-slot kernels exist for K = 8, 12 and 16)
  if (!dense2 && g2.kind == KMIX_GATHER) {
    if (g2.D <= 4) d2t = g2.D == 3 ? 4 : g2.D;
    else if (KT == 8 || KT == 12 || KT == 16) d2t = 8;
  }
  // a fused gather Mix1 with the same neighbour count as Mix2 (both mixes on one topology, as in
  // the paper's LocalM1M2) also gets a static gather
  const bool same_d1 = a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER && d2t > 0 &&
                       (g1.D == d2t || (g1.D == 3 && d2t == 4) || (g1.D > 4 && d2t == 8));
  auto go = [&]<int KTc, int VECc, int Cc, int D2c, bool SAME1>() -> int {
    int grid = 0;
    constexpr bool kPadBuilt = KTc == 6 || KTc == 8 || KTc == 12 || KTc == 16;   // kernels that also exist zero-padded
    if constexpr (D2c == -2) {
      auto launch = [&](auto kern) -> int {
        if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
        kern<<<grid, Cc + 32, smem, st>>>(ta, d2, g1, tp, tl, tm, tx);
        return FGD_OK;
      };
      if constexpr (kPadBuilt) {
        if (pad) { if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, true, -1, -1, DenseMix, true>)) return r; }
        else if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, true, -1, -1, DenseMix>)) return r;
      } else {
        if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, true, -1, -1, DenseMix>)) return r;
      }
    } else {
      auto launch = [&](auto kern) -> int {
        if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
        kern<<<grid, Cc + 32, smem, st>>>(ta, g2, g1, tp, tl, tm, tx);
        return FGD_OK;
      };
      if constexpr (kPadBuilt) {
        if (pad) { if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, false, D2c, (SAME1 ? D2c : -1), GatherMix, true>)) return r; }
        else if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, false, D2c, (SAME1 ? D2c : -1), GatherMix>)) return r;
      } else {
        if (int r = launch(outer_step_tma_kernel<KTc, VECc, Cc, false, D2c, (SAME1 ? D2c : -1), GatherMix>)) return r;
      }
    }
    *grid_out = grid;
    return check_launch(c, "outer_step_tma_kernel");
  };
#define FGD_TMA_D(kt, v, cc, d)                                                             \
  return same_d1 ? go.template operator()<kt, v, cc, d, true>() : go.template operator()<kt, v, cc, d, false>();
#define FGD_TMA_CASE(kt, v, cc)                                                             \
  if (KT == kt && sh.vec == v && sh.consumers == cc) {                                      \
    if (dense2) return go.template operator()<kt, v, cc, -2, false>();                      \
    switch (d2t) {                                                                          \
      case 0: return go.template operator()<kt, v, cc, 0, false>();                         \
      case 1: FGD_TMA_D(kt, v, cc, 1)                                                       \
      case 2: FGD_TMA_D(kt, v, cc, 2)                                                       \
      case 4: FGD_TMA_D(kt, v, cc, 4)                                                       \
      default: return go.template operator()<kt, v, cc, -1, false>();                       \
    }                                                                                       \
  }
// the same plus the eight-slot kernels
#define FGD_TMA_CASE8(kt, v, cc)                                                            \
  if (KT == kt && sh.vec == v && sh.consumers == cc && !dense2 && d2t == 8) { FGD_TMA_D(kt, v, cc, 8) }  \
  FGD_TMA_CASE(kt, v, cc)
#if FGD_TMA_GROUP == 0
  FGD_TMA_CASE(0, 2, 256) FGD_TMA_CASE(0, 1, 256) FGD_TMA_CASE(0, 1, 128)
  FGD_TMA_CASE(2, 4, 256) FGD_TMA_CASE(2, 4, 128)
  FGD_TMA_CASE(4, 4, 256) FGD_TMA_CASE(4, 4, 128)
#elif FGD_TMA_GROUP == 1
  FGD_TMA_CASE8(8, 4, 256) FGD_TMA_CASE8(8, 4, 128)
  FGD_TMA_CASE(32, 1, 256) FGD_TMA_CASE(32, 1, 128)
#elif FGD_TMA_GROUP == 2
  FGD_TMA_CASE8(16, 2, 256) FGD_TMA_CASE8(16, 2, 128) FGD_TMA_CASE8(16, 1, 512)
  FGD_TMA_CASE(64, 1, 128)
#elif FGD_TMA_GROUP == 3
  FGD_TMA_CASE(3, 4, 256) FGD_TMA_CASE(3, 4, 128)
  FGD_TMA_CASE(6, 4, 256) FGD_TMA_CASE(6, 4, 128)
  FGD_TMA_CASE8(12, 2, 256) FGD_TMA_CASE8(12, 2, 128)
#endif
#undef FGD_TMA_CASE8
#undef FGD_TMA_CASE
#undef FGD_TMA_D
  return fail(c, FGD_ERR_UNSUPPORTED, "internal: no TMA kernel for this shape");
}

}  // namespace
