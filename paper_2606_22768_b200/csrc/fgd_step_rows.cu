// Fused outer step (Sec. 4.1 round equations / Algorithm 1, Nesterov update of App. B, consensus sums
// of Sec. 4.4) for a SPARSE Mix2 at any worker count, as a TMA-pipelined row gather.
//
// The column kernels give one thread all K rows of its columns, which needs the worker count at compile
// time; the tensor-core kernel runs 17..63 workers zero-padded to 32 / 48 / 64 and pays the larger shape's
// operand preparation whatever the mix.  Here the worker and neighbour-slot counts are run-time values:
// a producer thread streams K x 128 boxes of theta_prev, theta_local and the momentum (box height = K,
// nothing padded) into a ring of stages; each of eight consumer warps takes every eighth ROW of the tile,
// a lane owning four columns.  Per row: g of the row and of its Mix2 neighbours straight from the two
// staged boxes (16-byte shared-memory loads, indices and weights from a table in shared memory, uniform
// per warp), x from its source (a vector, a matrix, the gossip Mix1 gathered from the staged theta_prev,
// or the column mean of theta_prev), the update, two 16-byte stores.  What needs a whole column -- the
// mean of theta_new for the consensus sums and for next round's Mix1, the mean of theta_prev -- goes
// through one exchange of per-warp column sums in shared memory and one barrier among the consumers.
#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_kernels.cuh"
#include "fgd_tma_host.h"

using namespace fgd;

namespace {

constexpr int kRowWarps = 8, kRowConsumers = 32 * kRowWarps, kRowCols = 128, kRowMaxStages = 6;
constexpr int kRowF4 = kRowCols / 4;                         // float4 per staged row
constexpr size_t kRowStatic = 26 * 1024;                     // static shared memory: tables, exchange rows, barriers (25.2 KB)

__device__ __forceinline__ void rows_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ float4 f4_sub(const float4 a, const float4 b) {
  return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
}
__device__ __forceinline__ float4 f4_scale(const float s, const float4 a) {
  return make_float4(s * a.x, s * a.y, s * a.z, s * a.w);
}
__device__ __forceinline__ void f4_fma(float4& acc, const float s, const float4 a) {
  acc.x = fmaf(s, a.x, acc.x);
  acc.y = fmaf(s, a.y, acc.y);
  acc.z = fmaf(s, a.z, acc.z);
  acc.w = fmaf(s, a.w, acc.w);
}
__device__ __forceinline__ void f4_add(float4& acc, const float4 a) {
  acc.x += a.x;
  acc.y += a.y;
  acc.z += a.z;
  acc.w += a.w;
}
// Four columns starting at col of a row, zeros beyond P (whole: all four are inside).
__device__ __forceinline__ float4 ld_cols(const float* p, int64_t col, int64_t P, bool whole) {
  if (whole) {                                      // x is read once and never written here: past L1
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
  }
  float r[4];
#pragma unroll
  for (int t = 0; t < 4; ++t) r[t] = col + t < P ? p[t] : 0.f;
  return make_float4(r[0], r[1], r[2], r[3]);
}
__device__ __forceinline__ void st_cols(float* p, const float4 v, int64_t col, int64_t P, bool whole) {
  if (whole) {
    __stcs(reinterpret_cast<float4*>(p), v);
  } else {
    const float r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t)
      if (col + t < P) p[t] = r[t];
  }
}

// D2T / D1T: neighbour slots of Mix2 / of a fused gossip Mix1 as unrolled (1, 2, 4 or 8 >= the used
// count; unused slots point at the row itself with weight 0).  D1T = 0: Mix1 is not a gossip mix.
// RPW: rows per warp, 8 (any worker count, one CTA per SM) or 4 (up to 32 workers: half the registers, so
// that two CTAs share an SM where two of their two-stage rings fit -- with few rows a tile is short and its
// fixed chain of waits, one CTA's worth, would otherwise show).
template <int D2T, int D1T, int RPW>
__global__ void __launch_bounds__(kRowConsumers + 32, RPW == 4 ? 2 : 1)
outer_step_rows_kernel(const TmaStepArgs ta, const GatherMix m2, const GatherMix m1,
                       const __grid_constant__ CUtensorMap tm_prev, const __grid_constant__ CUtensorMap tm_local,
                       const __grid_constant__ CUtensorMap tm_mom) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kRowMaxStages];
  __shared__ int abort_flag;
  __shared__ int s_n2[FGD_MAX_K * FGD_MAX_D], s_n1[D1T > 0 ? FGD_MAX_K * FGD_MAX_D : 1];   // float4 index of the neighbour's row
  __shared__ float s_w2[FGD_MAX_K * FGD_MAX_D], s_w1[D1T > 0 ? FGD_MAX_K * FGD_MAX_D : 1];
  __shared__ float s_ws2[FGD_MAX_K], s_ws1[D1T > 0 ? FGD_MAX_K : 1];
  // per-warp column sums, [tile parity][0: theta_new, 1: theta_prev][warp][column]
  __shared__ __align__(16) float xch[2][2][kRowWarps][kRowCols];
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  const StepArgs& a = ta.s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = a.K, STAGES = ta.stages;
  const uint32_t BOX = (uint32_t)K * kRowCols * 4, STAGE = 3 * BOX;
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + kRowCols - 1) / kRowCols;
  const bool want_cd = a.partials != nullptr;
  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[kRowMaxStages + s]), kRowWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < K * FGD_MAX_D; i += blockDim.x) {
    s_n2[i] = m2.nbr[i] * kRowF4;
    s_w2[i] = m2.w[i];
    if constexpr (D1T > 0) {
      s_n1[i] = m1.nbr[i] * kRowF4;
      s_w1[i] = m1.w[i];
    }
  }
  for (int i = tid; i < K; i += blockDim.x) {
    s_ws2[i] = m2.w_self[i];
    if constexpr (D1T > 0) s_ws1[i] = m1.w_self[i];
  }
  __syncthreads();

  double dacc[RPW];                       // consensus sums of rows warp, warp + 8, ... (this lane's columns)
#pragma unroll
  for (int r = 0; r < RPW; ++r) dacc[r] = 0.0;

  if (warp == kRowWarps) {
    // ===================================================== producer warp (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[kRowMaxStages + s]), (use - 1) & 1, ta.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        mbar_expect_tx(full, STAGE);
        if (i == ta.skip_tile) continue;             // test hook: these loads never arrive
        const uint32_t dst = smem_u32(base + (size_t)s * STAGE);
        const int c0 = (int)(tile * kRowCols);
        tma_load_2d(dst, &tm_prev, c0, 0, full, policy);
        tma_load_2d(dst + BOX, &tm_local, c0, 0, full, policy);
        tma_load_2d(dst + 2 * BOX, &tm_mom, c0, 0, full, policy);
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)     // never exit under a copy in flight
        if (j != ta.skip_tile) mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, ta.spin_limit);
    }
  } else {
    // ===================================================== consumers
    const float lr = a.lr, mu = a.mu, invK = 1.0f / (float)K;
    const bool x_vector = a.xsrc == XSRC_VECTOR, x_matrix = a.xsrc == XSRC_MATRIX;
    const bool x_mean = a.xsrc == XSRC_FUSED && m1.kind == KMIX_MEAN;
    const bool need_mean = want_cd || a.x_next != nullptr;     // the column mean of theta_new
    // From four Mix2 slots on, g = theta_prev - theta_local is formed once per row, in place over the
    // theta_local box, and the gather reads one box instead of two (D2T + 4 loads per row instead of 2 D2T + 2).
    constexpr bool PRE = D2T >= 4;
    const bool has_barrier = need_mean || x_mean || PRE;
    // x from global memory (a vector or a matrix) is fetched one tile ahead into registers: its latency
    // would otherwise stand at the head of every tile (x per column: 4.5 -> 5.7 TB/s at 33 workers)
    float4 xv_next = make_float4(0.f, 0.f, 0.f, 0.f), xm_next[RPW];
    auto fetch_x = [&](int64_t tile_) {
      const int64_t c_ = tile_ * kRowCols + 4 * lane;
      if (tile_ >= ntiles || c_ >= P) {              // columns outside the tensor count as zeros everywhere below
        xv_next = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 0; r < RPW; ++r) xm_next[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
      }
      const bool whole_ = c_ + 3 < P;
      if (x_vector) xv_next = ld_cols(a.x + c_, c_, P, whole_);
      if (x_matrix) {
#pragma unroll
        for (int r = 0; r < RPW; ++r)
          if (warp + kRowWarps * r < K) xm_next[r] = ld_cols(a.x + (size_t)(warp + kRowWarps * r) * ld + c_, c_, P, whole_);
      }
    };
#pragma unroll
    for (int r = 0; r < RPW; ++r) xm_next[r] = make_float4(0.f, 0.f, 0.f, 0.f);
    fetch_x(blockIdx.x);
    int64_t i = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
      const int s = (int)(i % STAGES), par = (int)(i & 1);
      float4 xc = xv_next, xm[RPW];         // x when it is one value per column / this warp's rows of a matrix x
#pragma unroll
      for (int r = 0; r < RPW; ++r) xm[r] = xm_next[r];
      fetch_x(tile + gridDim.x);
      const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[s]), (uint32_t)(i / STAGES) & 1, ta.spin_limit));
      if (!ok) {                                     // (taken per warp; the CTA-wide decision follows the barrier)
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
        if (!has_barrier) break;                     // no barrier in this configuration: nobody waits for this warp
      }
      const float4* A = reinterpret_cast<const float4*>(base + (size_t)s * STAGE) + lane;   // theta_prev
      float4* B = const_cast<float4*>(A) + (size_t)K * kRowF4;                              // theta_local (PRE: g)
      const float4* C = B + (size_t)K * kRowF4;                                             // momentum
      const int64_t col = tile * kRowCols + 4 * lane;
      const bool whole = col + 3 < P, any = col < P;
      const bool mixed = mix2_applies(a, col);       // subset option: Mix2 only inside the ranges
      if (x_mean) {
        xc = make_float4(0.f, 0.f, 0.f, 0.f);                                  // column mean of theta_prev: this warp's rows first
        float4 sp = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ok)
          for (int m = warp; m < K; m += kRowWarps) f4_add(sp, A[m * kRowF4]);
        *reinterpret_cast<float4*>(&xch[par][1][warp][4 * lane]) = sp;
        rows_bar_sync(1, kRowConsumers);
        if (*(volatile int*)&abort_flag) break;      // uniform: written before the barrier
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) f4_add(xc, *reinterpret_cast<const float4*>(&xch[par][1][w][4 * lane]));
        xc = f4_scale(invK, xc);
      }
      if constexpr (PRE) {
        if (ok)
          for (int m = warp; m < K; m += kRowWarps) B[m * kRowF4] = f4_sub(A[m * kRowF4], B[m * kRowF4]);
        rows_bar_sync(3, kRowConsumers);
        if (*(volatile int*)&abort_flag) break;      // uniform: written before the barrier
      }
      float4 tn[RPW];
      float4 colsum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        const int m = warp + kRowWarps * r;
        tn[r] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m < K && ok) {
          const size_t off = (size_t)m * ld + col;
          float4 x = x_matrix ? xm[r] : xc;
          const float4 tp = A[m * kRowF4];
          const float4 d0 = PRE ? B[m * kRowF4] : f4_sub(tp, B[m * kRowF4]);
          const float4 vv = C[m * kRowF4];
          float4 g = f4_scale(s_ws2[m], d0);
#pragma unroll
          for (int j = 0; j < D2T; ++j) {
            const int n = s_n2[m * FGD_MAX_D + j];
            f4_fma(g, s_w2[m * FGD_MAX_D + j], PRE ? B[n] : f4_sub(A[n], B[n]));
          }
          if (!mixed) g = d0;                        // identity Mix2 on this column group
          if constexpr (D1T > 0) {
            x = f4_scale(s_ws1[m], tp);
#pragma unroll
            for (int j = 0; j < D1T; ++j) f4_fma(x, s_w1[m * FGD_MAX_D + j], A[s_n1[m * FGD_MAX_D + j]]);
          }
          float4 vn, t;
          vn.x = fmaf(mu, vv.x, g.x); t.x = x.x - lr * fmaf(mu, vn.x, g.x);
          vn.y = fmaf(mu, vv.y, g.y); t.y = x.y - lr * fmaf(mu, vn.y, g.y);
          vn.z = fmaf(mu, vv.z, g.z); t.z = x.z - lr * fmaf(mu, vn.z, g.z);
          vn.w = fmaf(mu, vv.w, g.w); t.w = x.w - lr * fmaf(mu, vn.w, g.w);
          if (any) {
            st_cols(a.momentum + off, vn, col, P, whole);
            st_cols(a.theta_new + off, t, col, P, whole);
          }
          tn[r] = t;
          f4_add(colsum, t);
        }
      }
      if (need_mean) *reinterpret_cast<float4*>(&xch[par][0][warp][4 * lane]) = colsum;
      // (the in-place g rows were written through the generic proxy; the next TMA copy into this stage is not)
      if constexpr (PRE) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();                                  // every lane has read its part of the stage
      if (lane == 0 && ok) mbar_arrive(smem_u32(&bars[kRowMaxStages + s]));
      if (need_mean) {
        rows_bar_sync(2, kRowConsumers);
        if (*(volatile int*)&abort_flag) break;      // uniform: written before the barrier
        float4 mean = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < kRowWarps; ++w) f4_add(mean, *reinterpret_cast<const float4*>(&xch[par][0][w][4 * lane]));
        mean = f4_scale(invK, mean);
        if (a.x_next != nullptr && warp == 0 && any) st_cols(a.x_next + col, mean, col, P, whole);
        if (want_cd) {
#pragma unroll
          for (int r = 0; r < RPW; ++r) {
            if (warp + kRowWarps * r < K) {
              const float4 d = f4_sub(tn[r], mean);
              dacc[r] += (double)fmaf(d.x, d.x, fmaf(d.y, d.y, fmaf(d.z, d.z, d.w * d.w)));
            }
          }
        }
      } else if (!ok) {
        break;
      }
    }
  }

  // ---- consensus sums: every row belongs to one warp, so a warp-level reduction finishes it
  if (want_cd && warp < kRowWarps) {
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      const int m = warp + kRowWarps * r;
      double d = dacc[r];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
      if (lane == 0 && m < K) a.partials[(size_t)blockIdx.x * K + m] = d;
    }
  }
  if (want_cd) finalize_in_last_cta(a.partials, K, a.cd_out, a.done);
}

}  // namespace

// A sparse (or identity) Mix2 without the momentum-averaging option, TMA-compatible tensors.
bool fgd_step_rows_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2) {
  if (dense2 || g2.kind != KMIX_GATHER || a.avg_momentum) return false;
  if (!c->encode_tiled || c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  if (a.xsrc != XSRC_FUSED && !aligned16(a.x)) return false;
  if (a.x_next && !aligned16(a.x_next)) return false;
  const size_t stage = 3 * (size_t)c->K * kRowCols * 4;
  return (size_t)c->max_smem_optin >= 2 * stage + 128 + kRowStatic;
}

namespace {
int slot_class(int D) { return D <= 1 ? 1 : (D <= 2 ? 2 : (D <= 4 ? 4 : 8)); }
}  // namespace

int fgd_launch_step_rows(fgd_ctx* c, const StepArgs& a, const GatherMix& g2, const GatherMix& g1, cudaStream_t st,
                         int* grid_out) {
  CUtensorMap tp, tl, tm;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, kRowCols)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, kRowCols)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, kRowCols)) return rc;
  const size_t stage = 3 * (size_t)c->K * kRowCols * 4;
  // one CTA per SM: as many stages as its shared memory holds; up to 28 workers two CTAs with two or three stages each
  const bool two_ctas = c->K <= 28;
  const size_t budget = two_ctas ? (size_t)c->max_smem_optin / 2 - 2048 : (size_t)c->max_smem_optin;
  int stages = (int)((budget - kRowStatic - 128) / stage);
  stages = stages < 2 ? 2 : (stages > kRowMaxStages ? kRowMaxStages : stages);
  const size_t smem = 128 + stages * stage;
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = 3;
  ta.stages = stages;
  ta.spin_limit = c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit;
  ta.skip_tile = c->dbg_skip_tile;
  const int64_t ntiles = (c->P + kRowCols - 1) / kRowCols;
  auto launch = [&](auto kern) -> int {
    if (int rc = persistent_grid(c, kern, kRowConsumers + 32, smem, ntiles, grid_out)) return rc;
    kern<<<*grid_out, kRowConsumers + 32, smem, st>>>(ta, g2, g1, tp, tl, tm);
    return check_launch(c, "outer_step_rows_kernel");
  };
  const bool gossip1 = a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER;
  const int d2 = slot_class(g2.D), d1 = gossip1 ? slot_class(g1.D) : 0;
#define FGD_CASE(x2, x1) \
  if (d2 == x2 && d1 == x1) return two_ctas ? launch(outer_step_rows_kernel<x2, x1, 4>) : launch(outer_step_rows_kernel<x2, x1, 8>);
  FGD_CASE(1, 0) FGD_CASE(2, 0) FGD_CASE(4, 0) FGD_CASE(8, 0)
  FGD_CASE(1, 1) FGD_CASE(2, 1) FGD_CASE(4, 1) FGD_CASE(8, 1)
  FGD_CASE(1, 2) FGD_CASE(2, 2) FGD_CASE(4, 2) FGD_CASE(8, 2)
  FGD_CASE(1, 4) FGD_CASE(2, 4) FGD_CASE(4, 4) FGD_CASE(8, 4)
  FGD_CASE(1, 8) FGD_CASE(2, 8) FGD_CASE(4, 8) FGD_CASE(8, 8)
#undef FGD_CASE
  return fail(c, FGD_ERR_UNSUPPORTED, "internal: no row-gather step kernel for %d / %d neighbour slots", g2.D, g1.D);
}
