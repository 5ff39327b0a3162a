// TMA-pipelined fused step, worker-count group 3: 3, 6 and 12 workers (see fgd_step_tma_launch.inl).
#define FGD_TMA_GROUP 3
#include "fgd_step_tma_launch.inl"

int fgd_launch_step_tma_g3(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                            const GatherMix& g1, FgdTmaShape shape, cudaStream_t st, int* grid_out) {
  return launch_step_tma_group(c, a, dense2, g2, d2, g1, TmaShape{shape.vec, shape.consumers, shape.stages}, st, grid_out);
}
