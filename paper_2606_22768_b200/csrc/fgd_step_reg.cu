// Register-path fused step compiled for the worker counts 17..31 (two columns per thread).
//
// These counts have no pipelined kernel of their own: the tensor-core kernel runs them zero-padded to
// 32 workers, which moves no extra HBM bytes but does the 32-worker shape's shared-memory traffic and
// operand preparation.  With every row index a compile-time constant the plain column kernel (one thread
// owns two columns of all K workers, g in thread-private shared-memory columns, theta_new and the
// consensus terms in registers) is the faster one up to the low twenties (see the choice in fgd_api.cu).
#include "fgd_ctx.h"
#include "fgd_kernels.cuh"
#include "fgd_step_tma.h"

namespace {

constexpr int kRegVec = 2;

template <int KT>
int launch_reg_k(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                 const GatherMix& g1, cudaStream_t st, int* grid) {
  const int64_t ntiles = (c->P + (int64_t)kBlock * kRegVec - 1) / ((int64_t)kBlock * kRegVec);
  const size_t col = sizeof(float) * (size_t)KT * kBlock * kRegVec;
  size_t smem = col + (a.stage_tp ? col : 0);
  if (dense2) {
    if (!StepTraits<KT, kRegVec, true>::kRegArrays) smem += col + sizeof(float) * (size_t)KT * kBlock;
    smem += sizeof(float) * (size_t)KT * KT;
    auto kern = outer_step_kernel<KT, kRegVec, true, kBlock, DenseMix>;
    if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, grid)) return r;
    kern<<<*grid, kBlock, smem, st>>>(a, d2, g1);
  } else {
    auto kern = outer_step_kernel<KT, kRegVec, false, kBlock, GatherMix>;
    if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, grid)) return r;
    kern<<<*grid, kBlock, smem, st>>>(a, g2, g1);
  }
  return check_launch(c, "outer_step_kernel");
}

}  // namespace

bool fgd_reg_k_built(int K) { return K >= 17 && K <= 31; }

int fgd_launch_step_reg_k(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                          const GatherMix& g1, cudaStream_t st, int* grid_out) {
  switch (c->K) {
#define FGD_CASE(k) case k: return launch_reg_k<k>(c, a, dense2, g2, d2, g1, st, grid_out);
    FGD_CASE(17) FGD_CASE(18) FGD_CASE(19) FGD_CASE(20) FGD_CASE(21) FGD_CASE(22) FGD_CASE(23) FGD_CASE(24)
    FGD_CASE(25) FGD_CASE(26) FGD_CASE(27) FGD_CASE(28) FGD_CASE(29) FGD_CASE(30) FGD_CASE(31)
#undef FGD_CASE
    default: return fail(c, FGD_ERR_UNSUPPORTED, "internal: no register kernel compiled for K = %d", c->K);
  }
}
