// Interface between the entry points and the TMA-pipelined fused-step launcher.
#ifndef FGD_STEP_TMA_H_
#define FGD_STEP_TMA_H_

#include <cuda_runtime.h>

#include "fgd_internal.h"

struct fgd_ctx;
struct FgdTmaShape {
  int vec, consumers, stages;
};
// Can the TMA kernel run this call?  Picks the tile shape.
// heavy: the call gathers a lot per column (see fgd_outer_step_ex); such calls run with twice the consumer warps.
bool fgd_tma_eligible(const fgd_ctx* c, const fgd::StepArgs& a, bool dense2, bool heavy, FgdTmaShape* out);
int fgd_launch_step_tma(fgd_ctx* c, const fgd::StepArgs& a, bool dense2, const fgd::GatherMix& g2,
                        const fgd::DenseMix& d2, const fgd::GatherMix& g1, FgdTmaShape shape, cudaStream_t st,
                        int* grid_out);
// Dense Mix2 on the tensor cores (17 <= K <= 64, padded to 32 / 48 / 64 workers).
bool fgd_tc_eligible(const fgd_ctx* c, const fgd::StepArgs& a, bool tc_at_32, const fgd::GatherMix& g1);
// Stand-alone mix on the tensor cores (dm holds the dense, transposed matrix of whatever mix it is).
bool fgd_mix_tc_eligible(const fgd_ctx* c, const float* in, bool really_dense);
int fgd_launch_mix_dense_tc(fgd_ctx* c, const float* in, float* out, const fgd::DenseMix& dm, cudaStream_t st);
int fgd_launch_step_dense_tc(fgd_ctx* c, const fgd::StepArgs& a, const fgd::DenseMix& d2, const fgd::GatherMix& g1,
                             cudaStream_t st, int* grid_out);
// Stand-alone sparse mix as a TMA-pipelined row gather, any worker and slot count (fgd_mix_gather_tma.cu).
bool fgd_mix_gather_tma_eligible(const fgd_ctx* c, const float* in, const float* out);
int fgd_launch_mix_gather_tma(fgd_ctx* c, const float* in, float* out, const fgd::GatherMix& gm, cudaStream_t st);
// Fused step with a sparse Mix2 as a TMA-pipelined row gather, any worker and slot count (fgd_step_rows.cu).
bool fgd_step_rows_eligible(const fgd_ctx* c, const fgd::StepArgs& a, bool dense2, const fgd::GatherMix& g2);
int fgd_launch_step_rows(fgd_ctx* c, const fgd::StepArgs& a, const fgd::GatherMix& g2, const fgd::GatherMix& g1,
                         cudaStream_t st, int* grid_out);
// Register-path fused step compiled for the worker counts 17..31 (fgd_step_reg.cu; two columns per thread).
bool fgd_reg_k_built(int K);
int fgd_launch_step_reg_k(fgd_ctx* c, const fgd::StepArgs& a, bool dense2, const fgd::GatherMix& g2, const fgd::DenseMix& d2,
                          const fgd::GatherMix& g1, cudaStream_t st, int* grid_out);
#endif
