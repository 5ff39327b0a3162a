// Stand-alone sparse mix out_m = w_self[m] in_m + sum_j w[m][j] in_nbr[m][j] (Sec. 3 definition of
// Mix_W with a gossip matrix), for any worker count, as a TMA-pipelined row gather.
//
// The column kernels (mix_kernel) keep all K rows of a thread's columns in registers on their way to
// thread-private shared-memory columns, which needs the worker count at compile time; above 16
// workers the counts without a kernel of their own ran on the tensor-core mix (2.2-5.4 TB/s, its
// per-tile chain does not get shorter with fewer rows) or on the 64-worker column kernel (4 TB/s).
// Here the worker count and the slot count are run-time values throughout: a producer thread streams
// K x 128 boxes into a ring of stages with 2-D TMA copies (box height = K, so nothing is padded),
// and each of eight consumer warps takes every eighth row of the tile -- one 16-byte shared-memory
// load per lane and neighbour slot, indices and weights from a small table in shared memory (uniform
// per warp), one 16-byte store per lane.  HBM traffic is the algorithmic 8 bytes per worker-parameter.
#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_tma_host.h"

using namespace fgd;

namespace {

constexpr int kGmConsumers = 256, kGmCols = 128, kGmMaxStages = 8;

struct GatherTmaArgs {
  float* out;
  int64_t P, ld;
  int K, stages;
  int* status;
  uint32_t spin_limit;
  int skip_tile;
};

// DT: compile-time neighbour slot count (-1 = read at run time).
template <int DT>
__global__ void __launch_bounds__(kGmConsumers + 32)
mix_gather_tma_kernel(const GatherTmaArgs a, const GatherMix gm, const __grid_constant__ CUtensorMap tm_in) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kGmMaxStages];
  __shared__ int abort_flag;
  __shared__ int s_nbr[FGD_MAX_K * FGD_MAX_D];     // float4 index of the neighbour's row in a stage
  __shared__ float s_w[FGD_MAX_K * FGD_MAX_D];
  __shared__ float s_ws[FGD_MAX_K];
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = a.K, STAGES = a.stages;
  const int D = DT >= 0 ? DT : gm.D;
  const uint32_t STAGE = (uint32_t)K * kGmCols * 4;
  const int64_t ntiles = (a.P + kGmCols - 1) / kGmCols;
  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[kGmMaxStages + s]), kGmConsumers / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < K * FGD_MAX_D; i += blockDim.x) {
    s_nbr[i] = gm.nbr[i] * (kGmCols / 4);
    s_w[i] = gm.w[i];
  }
  for (int i = tid; i < K; i += blockDim.x) s_ws[i] = gm.w_self[i];
  __syncthreads();

  if (warp == kGmConsumers / 32) {                 // ---- producer
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[kGmMaxStages + s]), (use - 1) & 1, a.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        mbar_expect_tx(full, STAGE);
        if (i == a.skip_tile) continue;              // test hook: these loads never arrive
        tma_load_2d(smem_u32(base + (size_t)s * STAGE), &tm_in, (int)(tile * kGmCols), 0, full, policy);
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)     // never exit under a copy in flight
        if (j != a.skip_tile) mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, a.spin_limit);
    }
    return;
  }

  // ---- consumers: warp w takes rows w, w + 8, ...; lane l takes columns 4 l .. 4 l + 3 of the tile
  int64_t i = 0;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
    const int s = (int)(i % STAGES);
    if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[s]), (uint32_t)(i / STAGES) & 1, a.spin_limit))) {
      *(volatile int*)&abort_flag = 1;
      atomicExch(a.status, FGD_ERR_TIMEOUT);
      break;
    }
    const float4* A = reinterpret_cast<const float4*>(base + (size_t)s * STAGE) + lane;
    const int64_t col = tile * kGmCols + 4 * lane;
    const bool whole = col + 3 < a.P;
#pragma unroll 2
    for (int m = warp; m < K; m += kGmConsumers / 32) {
      const float4 v = A[m * (kGmCols / 4)];
      const float ws = s_ws[m];
      float4 acc = make_float4(ws * v.x, ws * v.y, ws * v.z, ws * v.w);
      const int* nb = s_nbr + m * FGD_MAX_D;
      const float* wj = s_w + m * FGD_MAX_D;
#pragma unroll
      for (int j = 0; j < (DT >= 0 ? DT : FGD_MAX_D); ++j) {
        if (DT < 0 && j >= D) break;
        const float4 u = A[nb[j]];
        const float w = wj[j];
        acc.x = fmaf(w, u.x, acc.x);
        acc.y = fmaf(w, u.y, acc.y);
        acc.z = fmaf(w, u.z, acc.z);
        acc.w = fmaf(w, u.w, acc.w);
      }
      float* dst = a.out + (size_t)m * a.ld + col;
      if (whole) {
        __stcs(reinterpret_cast<float4*>(dst), acc);
      } else {
        const float r[4] = {acc.x, acc.y, acc.z, acc.w};
        for (int t = 0; t < 4; ++t)
          if (col + t < a.P) dst[t] = r[t];
      }
    }
    __syncwarp();                                    // every lane has read its part of the stage
    if (lane == 0) mbar_arrive(smem_u32(&bars[kGmMaxStages + s]));
  }
}

}  // namespace

bool fgd_mix_gather_tma_eligible(const fgd_ctx* c, const float* in, const float* out) {
  if (!c->encode_tiled || c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  return aligned16(in) && aligned16(out);
}

int fgd_launch_mix_gather_tma(fgd_ctx* c, const float* in, float* out, const GatherMix& gm, cudaStream_t st) {
  CUtensorMap tm;
  if (int rc = make_tensor_map(c, &tm, in, kGmCols)) return rc;
  const size_t stage = (size_t)c->K * kGmCols * 4;
  int stages = (int)((48 * 1024) / stage);           // four CTAs per SM (three at 33-64 workers: two stages of up to 32 KB)
  stages = stages < 2 ? 2 : (stages > kGmMaxStages ? kGmMaxStages : stages);
  const size_t smem = 128 + stages * stage;
  const int64_t ntiles = (c->P + kGmCols - 1) / kGmCols;
  const GatherTmaArgs a{out, c->P, c->ld, c->K, stages, c->status, c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit,
                        c->dbg_skip_tile};
  int grid = 0;
  auto launch = [&](auto kern) -> int {
    if (int rc = persistent_grid(c, kern, kGmConsumers + 32, smem, ntiles, &grid)) return rc;
    kern<<<grid, kGmConsumers + 32, smem, st>>>(a, gm, tm);
    return check_launch(c, "mix_gather_tma_kernel");
  };
  switch (gm.D) {
    case 0: return launch(mix_gather_tma_kernel<0>);
    case 1: return launch(mix_gather_tma_kernel<1>);
    case 2: return launch(mix_gather_tma_kernel<2>);
    case 3: case 4: return launch(mix_gather_tma_kernel<4>);
    default: return launch(mix_gather_tma_kernel<-1>);
  }
}
