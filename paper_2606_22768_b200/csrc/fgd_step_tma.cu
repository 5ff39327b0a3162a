// Host side of the TMA-pipelined fused outer step: eligibility, tensor maps, kernel selection.
#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_ctx.h"
#include "fgd_step_dense_tc.cuh"
#include "fgd_step_tma.cuh"
#include "fgd_step_tma.h"

using namespace fgd;

namespace {

// ---- TMA-pipelined fused step ------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D map of a [K, ld] fp32 matrix restricted to its first P columns; box = boxc columns x K rows.
// Columns at or beyond P read as zero.
int make_tensor_map(fgd_ctx* c, CUtensorMap* map, const float* base, int boxc) {
  const cuuint64_t dims[2] = {(cuuint64_t)c->P, (cuuint64_t)c->K};
  const cuuint64_t strides[1] = {(cuuint64_t)c->ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)boxc, (cuuint32_t)c->K};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(c, FGD_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return FGD_OK;
}

// Tensors per stage: theta_prev, theta_local, momentum, plus a matrix-valued Mix1 result only in
// the kernels that cannot keep it in registers (run-time K, dense Mix2 with K > 16).
int tma_n_tensors(const StepArgs& a, int KT, bool dense2) {
  const bool xregs = KT > 0 && !(dense2 && KT > 16);
  return (a.xsrc == XSRC_MATRIX && !xregs) ? 4 : 3;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tile shapes of the TMA kernel.  A stage holds n_tensors x K x (consumers * vec) floats and at
// least two stages must fit in shared memory; measured on B200, 256 consumer threads with
// K * vec = 32 (a 96 KB stage, two stages) is the fastest shape, narrower tiles are the
// fall-back when the Mix1 result is a staged matrix (four tensors per stage).
struct TmaShape {
  int vec, consumers, stages;
};
const int kTmaShapes[][3] = {  // {KT, vec, consumers}, in order of preference per KT
    {0, 1, 128},
    {2, 4, 256}, {2, 4, 128},
    {4, 4, 256}, {4, 4, 128},
    {8, 4, 256}, {8, 4, 128},
    {16, 2, 256}, {16, 2, 128},
    {32, 1, 256}, {32, 1, 128},
    {64, 1, 128},
};

size_t tma_fixed_smem(int K, int KT, bool dense2, int consumers) {
  return 128 + (dense2 ? sizeof(float) * K * K : 0) + (KT == 0 ? sizeof(float) * K * consumers : 0);
}

// Can the TMA kernel run this call?  Picks the tile shape.
bool tma_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, TmaShape* out) {
  if (!c->encode_tiled) return false;
  if (c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  if (a.xsrc == XSRC_MATRIX && !aligned16(a.x)) return false;
  const int K = c->K, KT = kt_of(K), NT = tma_n_tensors(a, KT, dense2);
  const size_t budget = (size_t)c->max_smem_optin - 4096;  // static shared memory + slack
  for (const auto& sh : kTmaShapes) {
    if (sh[0] != KT) continue;
    const int vec = sh[1], consumers = sh[2];
    if (a.xsrc == XSRC_VECTOR && (reinterpret_cast<uintptr_t>(a.x) % (sizeof(float) * vec)) != 0) continue;
    const size_t fixed = tma_fixed_smem(K, KT, dense2, consumers);
    const size_t stage = tma_stage_bytes(K, consumers * vec, NT);
    if (budget < fixed + 2 * stage) continue;
    int stages = (int)((budget - fixed) / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    *out = {vec, consumers, stages};
    return true;
  }
  return false;
}

int launch_step_tma(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                    const GatherMix& g1, TmaShape sh, cudaStream_t st, int* grid_out) {
  const int K = c->K, KT = kt_of(K);
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = tma_n_tensors(a, KT, dense2);
  ta.stages = sh.stages;
  const int T = sh.consumers * sh.vec;
  const int boxc = T < 256 ? T : 256;
  CUtensorMap tp, tl, tm, tx;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tx, a.xsrc == XSRC_MATRIX ? a.x : a.theta_prev, boxc)) return rc;
  const size_t smem = tma_fixed_smem(K, KT, dense2, sh.consumers) + tma_stage_bytes(K, T, ta.n_tensors) * sh.stages;
  const int64_t ntiles = (c->P + T - 1) / T;
  // neighbour count of a gather Mix2 as a template argument when it is one of the common ones
  // (identity 0, one-peer / matching 1, ring 2, hypercube of 16 workers 4); else read at run time
  int d2t = -1;
  if (!dense2 && g2.kind == KMIX_GATHER && (g2.D == 0 || g2.D == 1 || g2.D == 2 || g2.D == 4)) d2t = g2.D;
  // a fused gather Mix1 with the same neighbour count as Mix2 (both mixes on one topology, as in
  // the paper's LocalM1M2) also gets a static gather
  const bool same_d1 = a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER && d2t > 0 && g1.D == d2t;
  auto go = [&]<int KTc, int VECc, int Cc, int D2c, bool SAME1>() -> int {
    int grid = 0;
    if constexpr (D2c == -2) {
      auto kern = outer_step_tma_kernel<KTc, VECc, Cc, true, -1, -1, DenseMix>;
      if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
      kern<<<grid, Cc + 32, smem, st>>>(ta, d2, g1, tp, tl, tm, tx);
    } else {
      auto kern = outer_step_tma_kernel<KTc, VECc, Cc, false, D2c, (SAME1 ? D2c : -1), GatherMix>;
      if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
      kern<<<grid, Cc + 32, smem, st>>>(ta, g2, g1, tp, tl, tm, tx);
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
  FGD_TMA_CASE(0, 1, 128)
  FGD_TMA_CASE(2, 4, 256) FGD_TMA_CASE(2, 4, 128)
  FGD_TMA_CASE(4, 4, 256) FGD_TMA_CASE(4, 4, 128)
  FGD_TMA_CASE(8, 4, 256) FGD_TMA_CASE(8, 4, 128)
  FGD_TMA_CASE(16, 2, 256) FGD_TMA_CASE(16, 2, 128)
  FGD_TMA_CASE(32, 1, 256) FGD_TMA_CASE(32, 1, 128)
  FGD_TMA_CASE(64, 1, 128)
#undef FGD_TMA_CASE
#undef FGD_TMA_D
  return fail(c, FGD_ERR_UNSUPPORTED, "internal: no TMA kernel for this shape");
}

}  // namespace

// Tensor-core dense step: K = 64, Mix1 given as the averaged row or fused as a mean.
bool fgd_tc_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g1) {
  if (!dense2 || c->K != kTcK || !c->encode_tiled || a.n_ranges != 0) return false;
  if (c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  if (!(a.xsrc == XSRC_VECTOR || (a.xsrc == XSRC_FUSED && g1.kind == KMIX_MEAN))) return false;
  return (size_t)c->max_smem_optin >= kTcSmem + 2048;
}

int fgd_launch_step_dense_tc(fgd_ctx* c, const StepArgs& a, const DenseMix& d2, const GatherMix& g1, cudaStream_t st,
                             int* grid_out) {
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = 3;
  ta.stages = kTcStages;
  CUtensorMap tp, tl, tm;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, kTcCols)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, kTcCols)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, kTcCols)) return rc;
  const int64_t ntiles = (c->P + kTcCols - 1) / kTcCols;
  int grid = 0;
  auto kern = outer_step_dense_tc_kernel;
  if (int r = persistent_grid(c, kern, kTcConsumers + 32, kTcSmem, ntiles, &grid)) return r;
  kern<<<grid, kTcConsumers + 32, kTcSmem, st>>>(ta, d2, g1, tp, tl, tm);
  *grid_out = grid;
  return check_launch(c, "outer_step_dense_tc_kernel");
}

bool fgd_tma_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, FgdTmaShape* out) {
  TmaShape sh{0, 0, 0};
  if (!tma_eligible(c, a, dense2, &sh)) return false;
  out->vec = sh.vec;
  out->consumers = sh.consumers;
  out->stages = sh.stages;
  return true;
}

int fgd_launch_step_tma(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                        const GatherMix& g1, FgdTmaShape shape, cudaStream_t st, int* grid_out) {
  return launch_step_tma(c, a, dense2, g2, d2, g1, TmaShape{shape.vec, shape.consumers, shape.stages}, st, grid_out);
}
