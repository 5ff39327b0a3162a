// Fused outer step, TMA-pipelined variant (the fast path on sm_100a).
//
// The register-only kernel keeps every load it has in flight in registers, which caps the
// bytes in flight per SM well below what HBM3e needs.  Here one producer warp streams
// [K rows x T columns] boxes of theta_prev, theta_local and the momentum (and the Mix1 result
// when it is a matrix) into a ring of shared-memory stages with 2-D TMA loads
// (cp.async.bulk.tensor) that complete on mbarriers, so a full stage or more (~100-190 KB per
// SM) is always in flight regardless of register use.  Consumer threads each own VEC adjacent
// columns of the tile and walk all K rows in shared memory: every cross-worker quantity
// (neighbour gathers, column means) is thread-local, so consumers never synchronise with each
// other -- only with the producer, through the stage's full / empty mbarriers.  Results are
// streamed to HBM straight from registers.  Stage buffers are reused in place:
//     A = theta_prev tile, B = theta_local tile -> outer gradient g, C = momentum tile -> theta_new.
// Every mbarrier wait is bounded; on a timeout the kernel records FGD_ERR_TIMEOUT in the
// status word, drains its own copies and returns.
#ifndef FGD_STEP_TMA_CUH_
#define FGD_STEP_TMA_CUH_

#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_kernels.cuh"

namespace fgd {

constexpr uint32_t kSpinLimit = 1u << 24;  // try_wait iterations before a wait gives up (the launch may pass a smaller limit)

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait for the phase with the given parity; false = gave up after `limit` polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
      : "memory");
}
// Ask for a box of a tensor to be brought into L2 (no shared-memory destination, no completion).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int c0, int c1) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(c0), "r"(c1) : "memory");
}

struct TmaStepArgs {
  StepArgs s;
  int* status;       // device status word (0 = ok)
  int n_tensors;     // 3, or 4 when x is a [K, ld] matrix
  int stages;        // pipeline depth, 2..kMaxStages
  uint32_t spin_limit;  // polls before a bounded wait gives up (kSpinLimit unless a test shortened it)
  int skip_tile;     // test hook: the producer announces but does not issue the loads of each CTA's
                     // skip_tile-th tile, so that the consumers' wait runs out; -1 = off
};

// Shared-memory need of the kernel (bytes), also used by the host to size the launch.
__host__ __device__ inline size_t tma_stage_bytes(int K, int T, int n_tensors) {
  return (size_t)n_tensors * K * T * sizeof(float);
}

constexpr int kMaxStages = 8;

// D2T: compile-time neighbour count of a gather Mix2 (-1 = read at run time; ignored for a mean
// or dense Mix2).
// D1T: the same for a fused gather Mix1 (-1 = run time).
// PAD: the worker count KR = a.K is smaller than the compile-time KT and the problem is zero-padded
// to KT rows: the TMA boxes are KT rows tall (rows at or beyond KR lie outside the tensor and arrive
// as zeros without touching HBM), the padded rows of every mix carry zero weights, and loads of a
// matrix-valued x, all stores and the consensus terms are predicated on the row being real.  Worker
// counts 5, 7, 9-11 and 13-15 run this way on the 6, 8, 12 and 16-worker kernels.
template <int KT, int VEC, int CONSUMERS, bool DENSE2, int D2T, int D1T, typename M2, bool PAD = false>
// (for 3, 6 and 12 workers the compiler is told that one CTA per SM is all there will be -- the
// stage ring takes the shared memory -- which frees it from a self-imposed register target:
// K = 12 5.5 -> 6.2 TB/s; for the other counts the same hint measured 0-1.5 % slower)
__global__ void __launch_bounds__(CONSUMERS + 32, (KT == 3 || KT == 6 || KT == 12) ? 1 : 0)
outer_step_tma_kernel(const TmaStepArgs ta, const M2 m2, const GatherMix m1,
                      const __grid_constant__ CUtensorMap tm_prev, const __grid_constant__ CUtensorMap tm_local,
                      const __grid_constant__ CUtensorMap tm_mom, const __grid_constant__ CUtensorMap tm_x) {
  constexpr int T = CONSUMERS * VEC;          // columns per tile
  constexpr int BOXC = T < 256 ? T : 256;     // columns per TMA box (box extents are <= 256)
  constexpr int NBOX = T / BOXC;              // boxes per tensor per tile
  constexpr int TPB = BOXC / VEC;             // consumer threads per box
  constexpr int NWARP = CONSUMERS / 32 + 1;
  static_assert(T % BOXC == 0 && CONSUMERS % 32 == 0 && BOXC % VEC == 0, "tile must be whole TMA boxes");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kMaxStages];
  __shared__ int abort_flag;
  __shared__ double red[NWARP][FGD_MAX_K];

  const StepArgs& a = ta.s;
  const int K = KT > 0 ? KT : a.K;                 // rows of a tile
  const int KR = PAD ? a.K : K;                    // real workers (<= K)
  static_assert(!PAD || KT > 0, "padding needs a compile-time worker count");
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool want_cd = a.partials != nullptr;
  const int NT = ta.n_tensors;
  const int STAGES = ta.stages;
  const size_t tens_floats = (size_t)K * T;                 // one tensor's box in a stage
  const size_t stage_floats = tens_floats * NT;
  // TMA destinations must be 128-byte aligned: round the ring's start up (the launch adds 128 B)
  float* stages = reinterpret_cast<float*>(smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u));
  float* wts = stages + stage_floats * STAGES;              // dense Wt [K*K] (DENSE2 only)
  float* sas = wts + (DENSE2 ? K * K : 0);                  // runtime-K consensus sums [K][CONSUMERS]

  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + T - 1) / T;
  const size_t box_floats = (size_t)K * BOXC;               // one TMA box

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);                       // full: one expect_tx arrival
      mbar_init(smem_u32(&bars[kMaxStages + s]), CONSUMERS);      // empty: every consumer arrives
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if constexpr (DENSE2) {
    if constexpr (PAD) {                            // m2.Wt is packed with stride KR: zero rows / columns beyond it
      for (int i = tid; i < K * K; i += CONSUMERS + 32) {
        const int n = i / K, m = i % K;
        wts[i] = (n < KR && m < KR) ? m2.Wt[n * KR + m] : 0.f;
      }
    } else {
      for (int i = tid; i < K * K; i += CONSUMERS + 32) wts[i] = m2.Wt[i];
    }
  }
  __syncthreads();

  constexpr int KS = KT > 0 ? KT : 1;
  float sacc[KS];
#pragma unroll
  for (int m = 0; m < KS; ++m) sacc[m] = 0.f;

  if (warp == CONSUMERS / 32) {
    // ===================================================== producer warp (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[kMaxStages + s]), (use - 1) & 1, ta.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        const int64_t c0 = tile * T;
        const int64_t left = P - c0;                                  // > 0
        const int nbox = left >= T ? NBOX : (int)((left + BOXC - 1) / BOXC);   // boxes that touch the tensor
        mbar_expect_tx(full, (uint32_t)(box_floats * sizeof(float)) * (uint32_t)(nbox * NT));
        if (i == ta.skip_tile) continue;                              // test hook: these loads never arrive
        const uint32_t dst = smem_u32(stages + stage_floats * s);
        for (int b = 0; b < nbox; ++b) {
          const uint32_t d = dst + (uint32_t)(box_floats * sizeof(float)) * b;
          const int c = (int)(c0 + (int64_t)b * BOXC);
          tma_load_2d(d, &tm_prev, c, 0, full, policy);
          tma_load_2d(d + (uint32_t)(tens_floats * 4), &tm_local, c, 0, full, policy);
          tma_load_2d(d + (uint32_t)(tens_floats * 8), &tm_mom, c, 0, full, policy);
          if (NT == 4) tma_load_2d(d + (uint32_t)(tens_floats * 12), &tm_x, c, 0, full, policy);
        }
      }
      if (!ok) {   // give up: flag it
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      // The CTA must not exit under a copy that is still in flight (the consumers may have given up
      // early): wait, bounded, for the last use of every stage.  In a healthy run these have landed.
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)
        if (j != ta.skip_tile) mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, ta.spin_limit);
    }
  } else {
    // ===================================================== consumers
    if constexpr (KT == 0) {
      for (int m = 0; m < K; ++m) sas[m * CONSUMERS + tid] = 0.f;
    }
    const float invK = 1.0f / (float)KR;
    const float lr = a.lr, mu = a.mu;
    // A matrix-valued Mix1 result is used only by the thread that owns the column, so with a
    // compile-time K it is not staged: each thread prefetches its K rows of the NEXT tile
    // straight into registers while it works on the current one (a whole tile of lead time).
    constexpr bool XREGS = (KT > 0) && !(DENSE2 && KT > 16);
    constexpr int KX = XREGS ? KT : 1;
    const bool x_direct = XREGS && a.xsrc == XSRC_MATRIX;
    Pack<VEC> xr[KX], xr_next[KX];
    auto fetch_x = [&](int64_t tile_, Pack<VEC> (&dst)[KX]) {
      const int64_t c_ = tile_ * T + (int64_t)tid * VEC;
      if (tile_ < ntiles && c_ + VEC <= P) {
#pragma unroll
        for (int m = 0; m < KX; ++m) dst[m] = (!PAD || m < KR) ? ld_stream<VEC>(a.x + (size_t)m * ld + c_) : p_zero<VEC>();
      } else if (tile_ < ntiles && c_ < P) {
        for (int m = 0; m < KX; ++m)
          for (int q = 0; q < VEC; ++q) dst[m].v[q] = (c_ + q < P && (!PAD || m < KR)) ? a.x[(size_t)m * ld + c_ + q] : 0.f;
      }
    };
    if (x_direct) fetch_x(blockIdx.x, xr_next);
    int64_t i = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
      if (x_direct) {
#pragma unroll
        for (int m = 0; m < KX; ++m) xr[m] = xr_next[m];
        fetch_x(tile + gridDim.x, xr_next);
      }
      const int s = (int)(i % STAGES);
      const uint32_t use = (uint32_t)(i / STAGES);
      const int64_t col = tile * T + (int64_t)tid * VEC;
      const bool live = col < P;
      const bool whole = col + VEC <= P;       // false only for the one group that straddles P
      Pack<VEC> xv = p_zero<VEC>();
      if (a.xsrc == XSRC_VECTOR && live) {     // latency hides behind the wait
        if (whole) xv = ld_stream<VEC>(a.x + col);
        else
          for (int q = 0; q < VEC; ++q)
            if (col + q < P) xv.v[q] = a.x[col + q];
      }
      // (the give-up decision is taken per warp, so a warp never leaves the loop half way)
      if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[s]), use & 1, ta.spin_limit))) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
        break;
      }
      // this thread's box inside each tensor of the stage; within a box, element (m, t) of a
      // [K][TPB] array of Pack<VEC>
      float* A = stages + stage_floats * s + box_floats * (tid / TPB);   // theta_prev
      float* B = A + tens_floats;              // theta_local -> g
      float* C = B + tens_floats;              // momentum -> theta_new
      float* X = C + tens_floats;              // Mix1 result (matrix), if staged
      const int t = tid % TPB;
      if (live) {
        // With a compile-time K every per-worker value has a static register index, so all
        // shared-memory loads of a phase are issued before anything depends on them and
        // theta_new never goes back to shared memory.  (Runtime K keeps them in the stage.)
        constexpr bool REGS = (KT > 0) && !(DENSE2 && KT > 16);
        constexpr int KQ = REGS ? KT : 1;
        // ---- phase 1: outer gradients of all workers into B, column sums
        Pack<VEC> gsum = p_zero<VEC>(), tsum = p_zero<VEC>();
        const bool need_tsum = a.xsrc == XSRC_FUSED && m1.kind == KMIX_MEAN;
        if constexpr (REGS) {
          Pack<VEC> tpv[KQ], tlv[KQ];
#pragma unroll
          for (int m = 0; m < KQ; ++m) {
            tpv[m] = SCol<VEC>::ld(A, m * TPB + t);
            tlv[m] = SCol<VEC>::ld(B, m * TPB + t);
          }
#pragma unroll
          for (int m = 0; m < KQ; ++m) {
            const Pack<VEC> g = p_sub<VEC>(tpv[m], tlv[m]);
            gsum = p_add<VEC>(gsum, g);
            SCol<VEC>::st(B, m * TPB + t, g);
          }
          if (need_tsum) {
#pragma unroll
            for (int m = 0; m < KQ; ++m) tsum = p_add<VEC>(tsum, tpv[m]);
          }
        } else {
#pragma unroll 4
          for (int m = 0; m < K; ++m) {
            const Pack<VEC> tp = SCol<VEC>::ld(A, m * TPB + t);
            const Pack<VEC> tl = SCol<VEC>::ld(B, m * TPB + t);
            const Pack<VEC> g = p_sub<VEC>(tp, tl);
            gsum = p_add<VEC>(gsum, g);
            tsum = p_add<VEC>(tsum, tp);
            SCol<VEC>::st(B, m * TPB + t, g);
          }
        }
        if (a.xsrc != XSRC_VECTOR) xv = p_mul<VEC>(tsum, invK);   // fused mean Mix1
        const Pack<VEC> gmean = p_mul<VEC>(gsum, invK);
        Pack<VEC> asum = p_zero<VEC>();
        // ---- phase 2: mix, Nesterov step, stream out; theta_new stays in av[] (or in C)
        Pack<VEC> av[KQ];
        Pack<VEC> vbar = p_zero<VEC>();           // column mean of the momentum (GlobalM1S option)
        if constexpr (REGS) {
#pragma unroll
          for (int m = 0; m < KQ; ++m) av[m] = SCol<VEC>::ld(C, m * TPB + t);   // momentum, all rows
          if (a.avg_momentum) {
#pragma unroll
            for (int m = 0; m < KQ; ++m) vbar = p_add<VEC>(vbar, av[m]);
            vbar = p_mul<VEC>(vbar, invK);
#pragma unroll
            for (int m = 0; m < KQ; ++m) av[m] = vbar;
          }
        } else if (a.avg_momentum) {
          for (int m = 0; m < K; ++m) vbar = p_add<VEC>(vbar, SCol<VEC>::ld(C, m * TPB + t));
          vbar = p_mul<VEC>(vbar, invK);
        }
        const bool mixed = mix2_applies(a, col);   // subset option: Mix2 only inside the ranges
        float* const mom_col = a.momentum + col;
        float* const new_col = a.theta_new + col;
        auto finish_row = [&](int m, const Pack<VEC>& gh) {
          const size_t off = (size_t)m * ld;
          Pack<VEC> xm;
          if (a.xsrc == XSRC_MATRIX) {
            if constexpr (XREGS) xm = xr[m];
            else xm = SCol<VEC>::ld(X, m * TPB + t);
          } else if (a.xsrc == XSRC_FUSED && m1.kind == KMIX_GATHER) {
            xm = gather_row<VEC, TPB, D1T>(m1, m, A, t);
          } else {
            xm = xv;
          }
          Pack<VEC> v;
          if constexpr (REGS) v = av[m];
          else v = a.avg_momentum ? vbar : SCol<VEC>::ld(C, m * TPB + t);
          const Pack<VEC> vn = p_fma<VEC>(v, mu, gh);                       // v' = mu v + ghat
          const Pack<VEC> tn = p_fma<VEC>(p_fma<VEC>(vn, mu, gh), -lr, xm);   // x - lr (ghat + mu v')
          if (PAD && m >= KR) {                 // a padded row: nothing to store, nothing to count
            if constexpr (REGS) av[m] = p_zero<VEC>();
            return;
          }
          asum = p_add<VEC>(asum, tn);
          if (whole) {
            st_stream<VEC>(mom_col + off, vn);
            st_stream<VEC>(new_col + off, tn);
          } else {                              // columns at or beyond P exist only as zero fill
            for (int q = 0; q < VEC; ++q)
              if (col + q < P) {
                mom_col[off + q] = vn.v[q];
                new_col[off + q] = tn.v[q];
              }
          }
          if constexpr (REGS) av[m] = tn;
          else if (want_cd) SCol<VEC>::st(C, m * TPB + t, tn);
        };
        if (!mixed) {                               // identity Mix2 on this column group
#pragma unroll(KT > 0 ? KT : 2)
          for (int m = 0; m < K; ++m) finish_row(m, SCol<VEC>::ld(B, m * TPB + t));
        } else if constexpr (DENSE2) {
          dense_rows<KT, VEC, TPB, (KT > 0 && KT <= 16)>(K, wts, B, t, finish_row);
        } else {
#pragma unroll(KT > 0 ? KT : 2)
          for (int m = 0; m < K; ++m) {
            Pack<VEC> gh;
            if (m2.kind == KMIX_MEAN) gh = gmean;
            else gh = gather_row<VEC, TPB, D2T>(m2, m, B, t);
            finish_row(m, gh);
          }
        }
        if (a.x_next) {                             // next round's global-average Mix1, for free
          const Pack<VEC> xn = p_mul<VEC>(asum, invK);
          if (whole) st_stream<VEC>(a.x_next + col, xn);
          else
            for (int q = 0; q < VEC; ++q)
              if (col + q < P) a.x_next[col + q] = xn.v[q];
        }
        // ---- phase 3: squared deviation of theta_new from its column mean
        if (want_cd) {
          const Pack<VEC> nmean = p_mul<VEC>(asum, -invK);
#pragma unroll(KT > 0 ? KT : 4)
          for (int m = 0; m < K; ++m) {
            Pack<VEC> tv;
            if constexpr (REGS) tv = av[m];
            else tv = SCol<VEC>::ld(C, m * TPB + t);
            Pack<VEC> d = p_add<VEC>(tv, nmean);
            if (!whole) {
#pragma unroll
              for (int q = 0; q < VEC; ++q)
                if (col + q >= P) d.v[q] = 0.f;
            }
            const float sq = p_hsum<VEC>(p_fma<VEC>(d, d, p_zero<VEC>()));      // (sums of padded rows are never read)
            if constexpr (KT > 0) sacc[m] += sq;
            else sas[m * CONSUMERS + tid] += sq;
          }
        }
      }
      // this thread's reads and writes of the stage are done: order them before the TMA refill
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&bars[kMaxStages + s]));
    }
  }

  // ---- consensus partial sums of the CTA (deterministic order); the producer warp adds zeros
  if (want_cd) {
    const bool consumer = warp < CONSUMERS / 32;
    if constexpr (KT > 0) {
#pragma unroll
      for (int m = 0; m < KT; ++m) {
        double d = consumer ? (double)sacc[m] : 0.0;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
        if (lane == 0) red[warp][m] = d;
      }
    } else {
      for (int m = 0; m < K; ++m) {
        double d = consumer ? (double)sas[m * CONSUMERS + tid] : 0.0;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
        if (lane == 0) red[warp][m] = d;
      }
    }
  }
  __syncthreads();
  if (want_cd && tid < KR) {
    double d = 0.0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) d += red[w][tid];
    a.partials[(size_t)blockIdx.x * KR + tid] = d;
  }
  if (want_cd) finalize_in_last_cta(a.partials, KR, a.cd_out, a.done);
}

}  // namespace fgd
#endif
