// Host-side helpers shared by the translation units that launch TMA-based kernels.
#ifndef FGD_TMA_HOST_H_
#define FGD_TMA_HOST_H_

#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_ctx.h"
#include "fgd_step_tma.cuh"
#include "fgd_step_tma.h"

namespace {

// ---- TMA-pipelined fused step ------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D map of a [K, ld] fp32 matrix restricted to its first P columns; box = boxc columns x K rows.
// Columns at or beyond P read as zero.  box_rows > K asks for a taller box: its rows at or beyond K
// lie outside the tensor and are filled with zeros too.
int make_tensor_map(fgd_ctx* c, CUtensorMap* map, const float* base, int boxc, int box_rows = 0) {
  const cuuint64_t dims[2] = {(cuuint64_t)c->P, (cuuint64_t)c->K};
  const cuuint64_t strides[1] = {(cuuint64_t)c->ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)boxc, (cuuint32_t)(box_rows > 0 ? box_rows : c->K)};
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
    {0, 2, 256}, {0, 1, 256}, {0, 1, 128},   // run-time K: widest tile whose two stages fit
    {2, 4, 256}, {2, 4, 128},
    {3, 4, 256}, {3, 4, 128},
    {4, 4, 256}, {4, 4, 128},
    {6, 4, 256}, {6, 4, 128},
    {8, 4, 256}, {8, 4, 128},
    {12, 2, 256}, {12, 2, 128},
    {16, 1, 512}, {16, 2, 256}, {16, 2, 128},   // 512 x 1: gather-heavy calls (see fgd_tma_eligible)
    {32, 1, 256}, {32, 1, 128},
    {64, 1, 128},
};

size_t tma_fixed_smem(int K, int KT, bool dense2, int consumers) {
  return 128 + (dense2 ? sizeof(float) * K * K : 0) + (KT == 0 ? sizeof(float) * K * consumers : 0);
}

// Can the TMA kernel run this call?  Picks the tile shape.
bool tma_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, bool heavy, TmaShape* out) {
  if (!c->encode_tiled) return false;
  if (c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  if (a.xsrc == XSRC_MATRIX && !aligned16(a.x)) return false;
  const int KT = kt_tma_of(c->K), K = KT > 0 ? KT : c->K, NT = tma_n_tensors(a, KT, dense2);   // K: rows of a tile (padded)
  const size_t budget = (size_t)c->max_smem_optin - 6144;  // static shared memory (barriers, reduction buffer) + slack
  for (const auto& sh : kTmaShapes) {
    if (sh[0] != KT) continue;
    if ((sh[2] == 512) != heavy) continue;   // 512 consumers: only, and always, for the gather-heavy calls
    const int vec = sh[1], consumers = sh[2];
    if (a.xsrc == XSRC_VECTOR && (reinterpret_cast<uintptr_t>(a.x) % (sizeof(float) * vec)) != 0) continue;
    if (a.x_next && (reinterpret_cast<uintptr_t>(a.x_next) % (sizeof(float) * vec)) != 0) continue;
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


}  // namespace
#endif
