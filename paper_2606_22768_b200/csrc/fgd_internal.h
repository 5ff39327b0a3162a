// Internal declarations shared by the host helpers and the CUDA launch code.
#ifndef FGD_INTERNAL_H_
#define FGD_INTERNAL_H_

#include <cstdarg>
#include <cstddef>
#include <cstdint>

#include "fgd.h"

namespace fgd {

extern thread_local char g_thread_error[256];
void set_thread_error(const char* fmt, ...);
uint64_t hash64(uint64_t seed, uint64_t round, uint64_t tag, uint64_t a, uint64_t b);
int validate_desc(const fgd_mix_desc* d, int K, char* msg, size_t msg_len);
void effective_weights(const fgd_mix_desc* d, double* w_eff, double* ws_eff);

// ---- what a kernel receives about a mix, passed BY VALUE as a kernel parameter (it lands
// in the constant bank, so the warp-uniform reads below are broadcast constant loads).
enum : int { KMIX_MEAN = 1, KMIX_GATHER = 2 };  // identity is a gather with D = 0, w_self = 1

struct GatherMix {
  int kind;                            // KMIX_MEAN or KMIX_GATHER
  int D;                               // used neighbour slots
  int nbr[FGD_MAX_K * FGD_MAX_D];      // row stride FGD_MAX_D; empty slots point at the row itself
  float w[FGD_MAX_K * FGD_MAX_D];      // effective weights (0 for dropped / empty slots)
  float w_self[FGD_MAX_K];             // effective self weights
};

struct DenseMix {
  float Wt[FGD_MAX_K * FGD_MAX_K];     // TRANSPOSED, packed with stride K: Wt[n*K+m] = W[m][n]
};

enum : int { XSRC_VECTOR = 0, XSRC_MATRIX = 1, XSRC_FUSED = 2 };

struct StepArgs {
  const float* theta_local;
  const float* theta_prev;
  float* momentum;
  float* theta_new;
  const float* x;       // XSRC_VECTOR: [P]; XSRC_MATRIX: [K, ld]; XSRC_FUSED: unused
  double* partials;     // [gridDim.x][K] consensus partial sums, or nullptr
  double* cd_out;       // [K] consensus sums, written by the CTA that finishes last (with partials)
  unsigned int* done;   // count of finished CTAs (zero between launches)
  int64_t P;
  int64_t ld;
  int K;
  int xsrc;
  int stage_tp;         // 1 when Mix1 is a fused gather (theta_prev columns staged in smem)
  float lr;
  float mu;
  // variants (fgd_outer_step_ex): Mix2 only inside column ranges; momentum averaged first
  int n_ranges;                          // 0 = Mix2 on every column
  int avg_momentum;                      // 1 = v_m <- mean_n v_n before the update
  float* x_next;                         // [P] or nullptr: column mean of theta_new (next round's global-average Mix1)
  int64_t range_lo[FGD_MAX_RANGES];
  int64_t range_hi[FGD_MAX_RANGES];
};

// Is Mix2 applied to the column group starting at `col`?  (Range bounds are multiples of 4
// columns, so a thread's group is never split.)
#ifdef __CUDACC__
__host__ __device__
#endif
inline bool mix2_applies(const StepArgs& a, int64_t col) {
  if (a.n_ranges == 0) return true;
  for (int i = 0; i < a.n_ranges; ++i)
    if (col >= a.range_lo[i] && col < a.range_hi[i]) return true;
  return false;
}

}  // namespace fgd
#endif
