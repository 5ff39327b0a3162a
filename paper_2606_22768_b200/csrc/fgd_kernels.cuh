// Device code of the outer-round kernels (sm_100a).
//
// Common design: HBM-streaming kernels in which ONE THREAD owns a group of VEC adjacent
// columns and walks all K worker rows of that group.  Everything that couples workers
// (neighbour gathers of Mix2 / Mix1, the column mean for global averaging and for the
// consensus distance) is therefore thread-local: no tile-wide barrier, no HBM scratch, and
// every tensor is read once and written once.  The per-worker values a thread needs to
// index with a RUNTIME worker id (the gathers) live in a thread-private column of shared
// memory laid out [m][thread] so that a warp's accesses are contiguous and conflict-free.
// Grids are persistent: a multiple of the SM count, tiles handed out round-robin so that
// concurrently running CTAs touch neighbouring columns of each row.
#ifndef FGD_KERNELS_CUH_
#define FGD_KERNELS_CUH_

#include <cuda_runtime.h>

#include "fgd_internal.h"

namespace fgd {

// ------------------------------------------------------------------ small vector helpers
template <int VEC>
struct Pack {
  float v[VEC];
};

template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_stream(const float* p);
template <>
__device__ __forceinline__ Pack<4> ld_stream<4>(const float* p) {
  const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
  return Pack<4>{{t.x, t.y, t.z, t.w}};
}
template <>
__device__ __forceinline__ Pack<2> ld_stream<2>(const float* p) {
  const float2 t = __ldcs(reinterpret_cast<const float2*>(p));
  return Pack<2>{{t.x, t.y}};
}
template <>
__device__ __forceinline__ Pack<1> ld_stream<1>(const float* p) {
  return Pack<1>{{__ldcs(p)}};
}

template <int VEC>
__device__ __forceinline__ void st_stream(float* p, const Pack<VEC>& a);
template <>
__device__ __forceinline__ void st_stream<4>(float* p, const Pack<4>& a) {
  __stcs(reinterpret_cast<float4*>(p), make_float4(a.v[0], a.v[1], a.v[2], a.v[3]));
}
template <>
__device__ __forceinline__ void st_stream<2>(float* p, const Pack<2>& a) {
  __stcs(reinterpret_cast<float2*>(p), make_float2(a.v[0], a.v[1]));
}
template <>
__device__ __forceinline__ void st_stream<1>(float* p, const Pack<1>& a) {
  __stcs(p, a.v[0]);
}

// thread-private shared-memory column: element (m, thread) of a [K][BLOCK] array of Pack<VEC>
template <int VEC>
struct SCol;
template <>
struct SCol<4> {
  typedef float4 T;
  static __device__ __forceinline__ Pack<4> ld(const float* base, int idx) {
    const float4 t = reinterpret_cast<const float4*>(base)[idx];
    return Pack<4>{{t.x, t.y, t.z, t.w}};
  }
  static __device__ __forceinline__ void st(float* base, int idx, const Pack<4>& a) {
    reinterpret_cast<float4*>(base)[idx] = make_float4(a.v[0], a.v[1], a.v[2], a.v[3]);
  }
};
template <>
struct SCol<2> {
  static __device__ __forceinline__ Pack<2> ld(const float* base, int idx) {
    const float2 t = reinterpret_cast<const float2*>(base)[idx];
    return Pack<2>{{t.x, t.y}};
  }
  static __device__ __forceinline__ void st(float* base, int idx, const Pack<2>& a) {
    reinterpret_cast<float2*>(base)[idx] = make_float2(a.v[0], a.v[1]);
  }
};
template <>
struct SCol<1> {
  static __device__ __forceinline__ Pack<1> ld(const float* base, int idx) {
    return Pack<1>{{base[idx]}};
  }
  static __device__ __forceinline__ void st(float* base, int idx, const Pack<1>& a) {
    base[idx] = a.v[0];
  }
};

// ---- element-wise helpers on Pack<VEC>.  For even VEC they use the packed fp32x2
// instructions of sm_100 (one issue slot for two lanes of the vector), which halves the
// floating-point instruction count of these issue-bound streaming kernels.
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_fma(const Pack<VEC>& a, float s, const Pack<VEC>& c) {  // a*s + c
  Pack<VEC> r;
  if constexpr (VEC % 2 == 0) {
#pragma unroll
    for (int i = 0; i < VEC; i += 2) {
      const float2 t = __ffma2_rn(make_float2(a.v[i], a.v[i + 1]), make_float2(s, s), make_float2(c.v[i], c.v[i + 1]));
      r.v[i] = t.x;
      r.v[i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC; ++i) r.v[i] = fmaf(a.v[i], s, c.v[i]);
  }
  return r;
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_fma(const Pack<VEC>& a, const Pack<VEC>& b, const Pack<VEC>& c) {  // a*b + c
  Pack<VEC> r;
  if constexpr (VEC % 2 == 0) {
#pragma unroll
    for (int i = 0; i < VEC; i += 2) {
      const float2 t = __ffma2_rn(make_float2(a.v[i], a.v[i + 1]), make_float2(b.v[i], b.v[i + 1]),
                                  make_float2(c.v[i], c.v[i + 1]));
      r.v[i] = t.x;
      r.v[i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC; ++i) r.v[i] = fmaf(a.v[i], b.v[i], c.v[i]);
  }
  return r;
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_add(const Pack<VEC>& a, const Pack<VEC>& b) {
  Pack<VEC> r;
  if constexpr (VEC % 2 == 0) {
#pragma unroll
    for (int i = 0; i < VEC; i += 2) {
      const float2 t = __fadd2_rn(make_float2(a.v[i], a.v[i + 1]), make_float2(b.v[i], b.v[i + 1]));
      r.v[i] = t.x;
      r.v[i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC; ++i) r.v[i] = a.v[i] + b.v[i];
  }
  return r;
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_mul(const Pack<VEC>& a, float s) {
  Pack<VEC> r;
  if constexpr (VEC % 2 == 0) {
#pragma unroll
    for (int i = 0; i < VEC; i += 2) {
      const float2 t = __fmul2_rn(make_float2(a.v[i], a.v[i + 1]), make_float2(s, s));
      r.v[i] = t.x;
      r.v[i + 1] = t.y;
    }
  } else {
#pragma unroll
    for (int i = 0; i < VEC; ++i) r.v[i] = a.v[i] * s;
  }
  return r;
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_sub(const Pack<VEC>& a, const Pack<VEC>& b) {  // a - b (exact: b * -1 + a)
  return p_fma<VEC>(b, -1.0f, a);
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> p_zero() {
  Pack<VEC> r;
#pragma unroll
  for (int i = 0; i < VEC; ++i) r.v[i] = 0.f;
  return r;
}
template <int VEC>
__device__ __forceinline__ float p_hsum(const Pack<VEC>& a) {
  float s = a.v[0];
#pragma unroll
  for (int i = 1; i < VEC; ++i) s += a.v[i];
  return s;
}

// Gather of a mix row from a thread-private shared column:
//   out = w_self[m] * col[m] + sum_{j < D} w[m][j] * col[nbr[m][j]]
// DT >= 0: the number of neighbour slots is a compile-time constant (fully unrolled, every
// index and weight a constant-bank operand, loads of all rows schedulable together);
// DT < 0: D is read at run time (warp-uniform loop).
template <int VEC, int BLOCK, int DT = -1>
__device__ __forceinline__ Pack<VEC> gather_row(const GatherMix& mx, int m, const float* col, int tid) {
  Pack<VEC> acc = p_mul<VEC>(SCol<VEC>::ld(col, m * BLOCK + tid), mx.w_self[m]);
  if constexpr (DT >= 0) {
#pragma unroll
    for (int j = 0; j < DT; ++j)
      acc = p_fma<VEC>(SCol<VEC>::ld(col, mx.nbr[m * FGD_MAX_D + j] * BLOCK + tid), mx.w[m * FGD_MAX_D + j], acc);
  } else {
    const int D = mx.D;
#pragma unroll 1
    for (int j = 0; j < D; ++j)
      acc = p_fma<VEC>(SCol<VEC>::ld(col, mx.nbr[m * FGD_MAX_D + j] * BLOCK + tid), mx.w[m * FGD_MAX_D + j], acc);
  }
  return acc;
}

// Deterministic block reduction of per-thread per-worker sums into partials[blockIdx.x][K].
// acc(m) returns this thread's fp32 sum for worker m; sums continue in fp64.
template <int BLOCK, typename AccFn>
__device__ __forceinline__ void block_reduce_partials(int K, AccFn acc, double* partials) {
  __shared__ double red[BLOCK / 32][FGD_MAX_K];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int m = 0; m < K; ++m) {
    double d = (double)acc(m);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
    if (lane == 0) red[warp][m] = d;
  }
  __syncthreads();
  if (threadIdx.x < K) {
    double d = 0.0;
#pragma unroll
    for (int w = 0; w < BLOCK / 32; ++w) d += red[w][threadIdx.x];
    partials[(size_t)blockIdx.x * K + threadIdx.x] = d;
  }
}

// Second stage of the consensus sums, inside the producing kernel: every thread of every CTA calls
// this after the CTA's row of partials[gridDim.x][K] is written.  The CTA that arrives last adds
// the rows up -- one warp per worker, lanes stride the CTAs, then a shuffle tree: a fixed order,
// so the result does not depend on which CTA happens to be last -- writes out[0..K) and re-arms
// the counter for the next launch.  (out == nullptr: the caller reduces the partials itself.)
__device__ __forceinline__ void finalize_in_last_cta(const double* partials, int K, double* out, unsigned int* counter) {
  if (out == nullptr) return;
  __shared__ int is_last;
  __threadfence();                      // this CTA's partials are visible device-wide ...
  __syncthreads();
  if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) + 1u == gridDim.x);   // ... before it is counted
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const int lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int m = threadIdx.x >> 5; m < K; m += nwarps) {
    double d = 0.0;
    for (unsigned int b = lane; b < gridDim.x; b += 32) d += __ldcg(partials + (size_t)b * K + m);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
    if (lane == 0) out[m] = d;
  }
  if (threadIdx.x == 0) *counter = 0u;
}

// Same reduction for sums held in a register array (static indexing only).
template <int BLOCK, int KR>
__device__ __forceinline__ void block_reduce_regs(int K, const float (&sacc)[KR], double* partials) {
  __shared__ double red[BLOCK / 32][FGD_MAX_K];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int m = 0; m < KR; ++m) {
    double d = (double)sacc[m];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
    if (lane == 0) red[warp][m] = d;
  }
  __syncthreads();
  if (threadIdx.x < K) {
    double d = 0.0;
#pragma unroll
    for (int w = 0; w < BLOCK / 32; ++w) d += red[w][threadIdx.x];
    partials[(size_t)blockIdx.x * K + threadIdx.x] = d;
  }
}

// Dense mix of a thread-private column on the CUDA cores: for every row m,
//   out_m = sum_n W[m][n] * col[n],   W given transposed in shared memory (wts[n*K+m]).
// Rows are produced MB at a time so that one shared-memory read of col[n] feeds MB FMAs and
// the MB weights of a step are one or two 128-bit broadcast reads.  fn(m, out_m) consumes a row.
template <int KT, int VEC, int BLOCK, bool FULL_UNROLL, typename RowFn>
__device__ __forceinline__ void dense_rows(int K, const float* wts, const float* cols, int tid, RowFn fn) {
  constexpr int MB = (KT > 0 && KT < 8) ? KT : ((KT > 0 && KT % 8 != 0) ? 4 : 8);   // MB divides a compile-time K
  constexpr bool VECW = (KT > 0) && (KT % 4 == 0);   // rows of Wt are 16-byte aligned
#pragma unroll(FULL_UNROLL ? 8 : 1)
  for (int mb = 0; mb < K; mb += MB) {
    Pack<VEC> acc[MB];
#pragma unroll
    for (int r = 0; r < MB; ++r)
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[r].v[i] = 0.f;
#pragma unroll(FULL_UNROLL ? 16 : 4)
    for (int n = 0; n < K; ++n) {
      const Pack<VEC> gn = SCol<VEC>::ld(cols, n * BLOCK + tid);
      float w[MB];
      if constexpr (VECW) {
#pragma unroll
        for (int q = 0; q < MB / 4; ++q) {
          const float4 t = *reinterpret_cast<const float4*>(wts + n * K + mb + 4 * q);
          w[4 * q] = t.x; w[4 * q + 1] = t.y; w[4 * q + 2] = t.z; w[4 * q + 3] = t.w;
        }
      } else {
#pragma unroll
        for (int r = 0; r < MB; ++r) w[r] = (mb + r < K) ? wts[n * K + mb + r] : 0.f;
      }
#pragma unroll
      for (int r = 0; r < MB; ++r)
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[r].v[i] = fmaf(w[r], gn.v[i], acc[r].v[i]);
    }
#pragma unroll
    for (int r = 0; r < MB; ++r)
      if (mb + r < K) fn(mb + r, acc[r]);
  }
}

// ------------------------------------------------------------------ fused outer step
// One pass: g = theta_prev - theta_local; ghat = Mix2(g); x = Mix1 result (given or fused);
// v' = mu v + ghat; theta_new = x - lr (ghat + mu v'); optional consensus partial sums of
// theta_new.  Per worker-parameter: 12 B read (+4/K or +4 for a given x), 8 B written.
//
// KT      compile-time K (0 = runtime K, generic slow path)
// VEC     columns per thread (KT * VEC <= 64)
// DENSE2  Mix2 is a dense K x K matrix (M2 = DenseMix), else a mean / gather (M2 = GatherMix)
template <int KT, int VEC, bool DENSE2>
struct StepTraits {
  // per-worker theta_new values and consensus sums stay in registers when every index is a
  // compile-time constant; otherwise they live in thread-private shared columns.
  static constexpr bool kRegArrays = (KT > 0) && !(DENSE2 && KT > 16);
};

template <int KT, int VEC, bool DENSE2, int BLOCK, typename M2>
__global__ void __launch_bounds__(BLOCK)
outer_step_kernel(const StepArgs a, const M2 m2, const GatherMix m1) {
  typedef StepTraits<KT, VEC, DENSE2> TR;
  extern __shared__ __align__(16) float smem[];
  const int K = KT > 0 ? KT : a.K;
  const int tid = threadIdx.x;
  const bool want_cd = a.partials != nullptr;

  // shared-memory carve-up (floats)
  float* gs = smem;                                           // [K][BLOCK] Pack<VEC>: g columns
  float* tps = gs + (size_t)K * BLOCK * VEC;                  // same, theta_prev (if staged)
  float* avs = tps + (a.stage_tp ? (size_t)K * BLOCK * VEC : 0);   // theta_new (if !kRegArrays)
  float* sas = avs + (TR::kRegArrays ? 0 : (size_t)K * BLOCK * VEC);  // consensus sums (if !kRegArrays)
  float* wts = sas + (TR::kRegArrays ? 0 : (size_t)K * BLOCK);        // dense Wt [K*K]

  if constexpr (DENSE2) {
    for (int i = tid; i < K * K; i += BLOCK) wts[i] = m2.Wt[i];
  }
  constexpr int KR = TR::kRegArrays ? KT : 1;
  float sacc[KR];
#pragma unroll
  for (int m = 0; m < KR; ++m) sacc[m] = 0.f;
  if constexpr (!TR::kRegArrays) {
    for (int m = 0; m < K; ++m) sas[m * BLOCK + tid] = 0.f;
  }
  if constexpr (DENSE2) __syncthreads();

  const float invK = 1.0f / (float)K;
  const float lr = a.lr, mu = a.mu;
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + (int64_t)BLOCK * VEC - 1) / ((int64_t)BLOCK * VEC);

  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t col = (tile * BLOCK + tid) * VEC;
    if (col >= P) continue;

    // ---- phase 1: outer gradient of every worker into the private column, column sums.
    // With a compile-time K the momentum rows are requested here too: measured on B200, having
    // all 3K loads of a column group in flight at once is worth 3.2 -> 5.3 TB/s on this kernel.
    Pack<VEC> gsum = p_zero<VEC>(), tsum = p_zero<VEC>();
    Pack<VEC> vreg[KR];
#pragma unroll(KT > 0 ? KT : 4)
    for (int m = 0; m < K; ++m) {
      const size_t off = (size_t)m * ld + col;
      const Pack<VEC> tp = ld_stream<VEC>(a.theta_prev + off);
      const Pack<VEC> tl = ld_stream<VEC>(a.theta_local + off);
      if constexpr (TR::kRegArrays) vreg[m] = ld_stream<VEC>(a.momentum + off);
      const Pack<VEC> g = p_sub<VEC>(tp, tl);
      gsum = p_add<VEC>(gsum, g);
      tsum = p_add<VEC>(tsum, tp);
      SCol<VEC>::st(gs, m * BLOCK + tid, g);
      if (a.stage_tp) SCol<VEC>::st(tps, m * BLOCK + tid, tp);
    }
    Pack<VEC> xv;
    if (a.xsrc == XSRC_VECTOR) {
      xv = ld_stream<VEC>(a.x + col);
    } else {
#pragma unroll
      for (int i = 0; i < VEC; ++i) xv.v[i] = tsum.v[i] * invK;  // used when Mix1 is a fused mean
    }
    Pack<VEC> gmean;
#pragma unroll
    for (int i = 0; i < VEC; ++i) gmean.v[i] = gsum.v[i] * invK;

    // ---- phase 2: per worker, mix the gradient, take the Nesterov step, stream out
    Pack<VEC> av[KR];
    Pack<VEC> asum;
#pragma unroll
    for (int i = 0; i < VEC; ++i) asum.v[i] = 0.f;

    Pack<VEC> vbar = p_zero<VEC>();              // column mean of the momentum (GlobalM1S option)
    if (a.avg_momentum) {
      if constexpr (TR::kRegArrays) {
#pragma unroll
        for (int m = 0; m < KR; ++m) vbar = p_add<VEC>(vbar, vreg[m]);
      } else {
        for (int m = 0; m < K; ++m) vbar = p_add<VEC>(vbar, ld_stream<VEC>(a.momentum + (size_t)m * ld + col));
      }
      vbar = p_mul<VEC>(vbar, invK);
    }
    const bool mixed = mix2_applies(a, col);     // subset option: Mix2 only inside the ranges
    auto finish_row = [&](int m, const Pack<VEC>& gh) {
      const size_t off = (size_t)m * ld + col;
      Pack<VEC> xm;
      if (a.xsrc == XSRC_MATRIX) xm = ld_stream<VEC>(a.x + off);
      else if (a.xsrc == XSRC_FUSED && m1.kind == KMIX_GATHER) xm = gather_row<VEC, BLOCK>(m1, m, tps, tid);
      else xm = xv;
      Pack<VEC> v;
      if (a.avg_momentum) v = vbar;
      else if constexpr (TR::kRegArrays) v = vreg[m];
      else v = ld_stream<VEC>(a.momentum + off);
      Pack<VEC> vn, tn;
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        vn.v[i] = fmaf(mu, v.v[i], gh.v[i]);
        tn.v[i] = xm.v[i] - lr * fmaf(mu, vn.v[i], gh.v[i]);
        asum.v[i] += tn.v[i];
      }
      st_stream<VEC>(a.momentum + off, vn);
      st_stream<VEC>(a.theta_new + off, tn);
      if constexpr (TR::kRegArrays) av[m] = tn;
      else if (want_cd) SCol<VEC>::st(avs, m * BLOCK + tid, tn);
    };

    if (!mixed) {                                 // identity Mix2 on this column group
#pragma unroll(KT > 0 ? KT : 2)
      for (int m = 0; m < K; ++m) finish_row(m, SCol<VEC>::ld(gs, m * BLOCK + tid));
    } else if constexpr (DENSE2) {
      dense_rows<KT, VEC, BLOCK, TR::kRegArrays>(K, wts, gs, tid, finish_row);
    } else {
#pragma unroll(KT > 0 ? KT : 2)
      for (int m = 0; m < K; ++m) {
        Pack<VEC> gh;
        if (m2.kind == KMIX_MEAN) gh = gmean;
        else gh = gather_row<VEC, BLOCK>(m2, m, gs, tid);
        finish_row(m, gh);
      }
    }

    if (a.x_next) st_stream<VEC>(a.x_next + col, p_mul<VEC>(asum, invK));   // next round's global-average Mix1
    // ---- consensus distance of theta_new: squared deviation from the column mean
    if (want_cd) {
#pragma unroll(KT > 0 ? KT : 4)
      for (int m = 0; m < K; ++m) {
        Pack<VEC> t;
        if constexpr (TR::kRegArrays) t = av[m];
        else t = SCol<VEC>::ld(avs, m * BLOCK + tid);
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
          const float d = t.v[i] - asum.v[i] * invK;
          s = fmaf(d, d, s);
        }
        if constexpr (TR::kRegArrays) sacc[m] += s;
        else sas[m * BLOCK + tid] += s;
      }
    }
  }

  if (want_cd) {
    if constexpr (TR::kRegArrays) {
      block_reduce_regs<BLOCK, KR>(K, sacc, a.partials);
    } else {
      block_reduce_partials<BLOCK>(K, [&](int m) { return sas[m * BLOCK + tid]; }, a.partials);
    }
    finalize_in_last_cta(a.partials, K, a.cd_out, a.done);
  }
}

// ------------------------------------------------------------------ stand-alone mix
// out_m = sum_n W[m][n] in_n.  MEAN may write the single averaged row (out_is_vector).
struct MixArgs {
  const float* in;
  float* out;
  int64_t P;
  int64_t ld;
  int K;
  int out_is_vector;
};

// DT: compile-time neighbour slot count of a sparse mix (-1 = read at run time), see gather_row.
template <int KT, int VEC, bool DENSE, int BLOCK, typename MX, int DT = -1>
__global__ void __launch_bounds__(BLOCK) mix_kernel(const MixArgs a, const MX mx) {
  extern __shared__ __align__(16) float smem[];
  const int K = KT > 0 ? KT : a.K;
  const int tid = threadIdx.x;
  float* cs = smem;                                  // [K][BLOCK] Pack<VEC>
  float* wts = cs + (size_t)K * BLOCK * VEC;         // dense Wt
  if constexpr (DENSE) {
    for (int i = tid; i < K * K; i += BLOCK) wts[i] = mx.Wt[i];
    __syncthreads();
  }
  const float invK = 1.0f / (float)K;
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + (int64_t)BLOCK * VEC - 1) / ((int64_t)BLOCK * VEC);
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t col = (tile * BLOCK + tid) * VEC;
    if (col >= P) continue;
    bool is_mean = false;
    if constexpr (!DENSE) is_mean = (mx.kind == KMIX_MEAN);
    if (is_mean) {
      // pure load-and-add: nothing between the K loads, so they are all in flight together
      Pack<VEC> sum = p_zero<VEC>();
      if constexpr (KT > 0) {
        Pack<VEC> t[KT];
#pragma unroll
        for (int m = 0; m < KT; ++m) t[m] = ld_stream<VEC>(a.in + (size_t)m * ld + col);
#pragma unroll
        for (int m = 0; m < KT; ++m) sum = p_add<VEC>(sum, t[m]);
      } else {
#pragma unroll 4
        for (int m = 0; m < K; ++m) sum = p_add<VEC>(sum, ld_stream<VEC>(a.in + (size_t)m * ld + col));
      }
      sum = p_mul<VEC>(sum, invK);
      if (a.out_is_vector) {
        st_stream<VEC>(a.out + col, sum);
      } else {
#pragma unroll(KT > 0 ? KT : 4)
        for (int m = 0; m < K; ++m) st_stream<VEC>(a.out + (size_t)m * ld + col, sum);
      }
      continue;
    }
    // all rows of the column group into the private column (loads first, then the stores)
    if constexpr (KT > 0) {
      Pack<VEC> t[KT];
#pragma unroll
      for (int m = 0; m < KT; ++m) t[m] = ld_stream<VEC>(a.in + (size_t)m * ld + col);
#pragma unroll
      for (int m = 0; m < KT; ++m) SCol<VEC>::st(cs, m * BLOCK + tid, t[m]);
    } else {
#pragma unroll 4
      for (int m = 0; m < K; ++m) SCol<VEC>::st(cs, m * BLOCK + tid, ld_stream<VEC>(a.in + (size_t)m * ld + col));
    }
    if constexpr (DENSE) {
      dense_rows<KT, VEC, BLOCK, false>(K, wts, cs, tid, [&](int m, const Pack<VEC>& r) {
        st_stream<VEC>(a.out + (size_t)m * ld + col, r);
      });
    } else {
#pragma unroll(KT > 0 ? KT : 2)
      for (int m = 0; m < K; ++m)
        st_stream<VEC>(a.out + (size_t)m * ld + col, gather_row<VEC, BLOCK, DT>(mx, m, cs, tid));
    }
  }
}

// ------------------------------------------------------------------ outer gradient
// g = theta_prev - theta_local, element-wise over the [K, P] window of [K, ld] matrices.
template <int VEC, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
outer_grad_kernel(const float* __restrict__ theta_prev, const float* __restrict__ theta_local,
                  float* __restrict__ g, int K, int64_t P, int64_t ld) {
  const int64_t groups = (P + VEC - 1) / VEC;  // P % VEC == 0 on the vector path
  const int64_t total = groups * K;
  for (int64_t i = (int64_t)blockIdx.x * BLOCK + threadIdx.x; i < total; i += (int64_t)gridDim.x * BLOCK) {
    const int64_t m = i / groups, c = (i - m * groups) * VEC;
    const size_t off = (size_t)m * ld + c;
    const Pack<VEC> tp = ld_stream<VEC>(theta_prev + off);
    const Pack<VEC> tl = ld_stream<VEC>(theta_local + off);
    Pack<VEC> r;
#pragma unroll
    for (int j = 0; j < VEC; ++j) r.v[j] = tp.v[j] - tl.v[j];
    st_stream<VEC>(g + off, r);
  }
}

// ------------------------------------------------------------------ consensus distance
// partials[block][m] = sum over the block's columns of (theta[m][p] - mean_p)^2.
template <int KT, int VEC, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
consensus_kernel(const float* __restrict__ theta, double* __restrict__ partials, int Krt, int64_t P,
                 int64_t ld, double* __restrict__ out, unsigned int* done) {
  extern __shared__ __align__(16) float smem[];
  const int K = KT > 0 ? KT : Krt;
  const int tid = threadIdx.x;
  constexpr int KR = KT > 0 ? KT : 1;
  float sacc[KR];
#pragma unroll
  for (int m = 0; m < KR; ++m) sacc[m] = 0.f;
  float* cs = smem;                               // runtime-K path: [K][BLOCK] values
  float* sas = cs + (size_t)K * BLOCK * VEC;      // runtime-K path: [K][BLOCK] sums
  if constexpr (KT == 0) {
    for (int m = 0; m < K; ++m) sas[m * BLOCK + tid] = 0.f;
  }
  const float invK = 1.0f / (float)K;
  const int64_t ntiles = (P + (int64_t)BLOCK * VEC - 1) / ((int64_t)BLOCK * VEC);
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t col = (tile * BLOCK + tid) * VEC;
    if (col >= P) continue;
    Pack<VEC> sum;
#pragma unroll
    for (int i = 0; i < VEC; ++i) sum.v[i] = 0.f;
    Pack<VEC> t[KR];
#pragma unroll(KT > 0 ? KT : 4)
    for (int m = 0; m < K; ++m) {
      const Pack<VEC> u = ld_stream<VEC>(theta + (size_t)m * ld + col);
#pragma unroll
      for (int i = 0; i < VEC; ++i) sum.v[i] += u.v[i];
      if constexpr (KT > 0) t[m] = u;
      else SCol<VEC>::st(cs, m * BLOCK + tid, u);
    }
#pragma unroll(KT > 0 ? KT : 4)
    for (int m = 0; m < K; ++m) {
      Pack<VEC> u;
      if constexpr (KT > 0) u = t[m];
      else u = SCol<VEC>::ld(cs, m * BLOCK + tid);
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        const float d = u.v[i] - sum.v[i] * invK;
        s = fmaf(d, d, s);
      }
      if constexpr (KT > 0) sacc[m] += s;
      else sas[m * BLOCK + tid] += s;
    }
  }
  if constexpr (KT > 0) {
    __shared__ double red[BLOCK / 32][FGD_MAX_K];
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int m = 0; m < KR; ++m) {
      double d = (double)sacc[m];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
      if (lane == 0) red[warp][m] = d;
    }
    __syncthreads();
    if (tid < K) {
      double d = 0.0;
#pragma unroll
      for (int w = 0; w < BLOCK / 32; ++w) d += red[w][tid];
      partials[(size_t)blockIdx.x * K + tid] = d;
    }
  } else {
    block_reduce_partials<BLOCK>(K, [&](int m) { return sas[m * BLOCK + tid]; }, partials);
  }
  finalize_in_last_cta(partials, K, out, done);
}

// Many workers (K = 32, 64): one thread per column would hold K values and K sums, which leaves one
// block per SM and too few loads in flight (77 % of the copy roofline at K = 64).  Here SPLIT threads
// share a column group, each owning R = K / SPLIT rows -- the register picture of the K = 16 kernel
// -- and exchange only their partial column sums through shared memory (double-buffered by tile
// parity: one barrier per tile).
// PAD: the real worker count KR < KT is a run-time value (17..31 on the 32-worker shape, 33..63 on the
// 64-worker one): rows at or beyond KR are never loaded (they count as zeros in the column sum, which is
// divided by KR) and their sums are dropped.
template <int KT, int SPLIT, int VEC, int BLOCK, bool PAD = false>
__global__ void __launch_bounds__(BLOCK)
consensus_split_kernel(const float* __restrict__ theta, double* __restrict__ partials, int64_t P, int64_t ld,
                       double* __restrict__ out, unsigned int* done, int k_real = KT) {
  const int KR = PAD ? k_real : KT;
  constexpr int R = KT / SPLIT;      // rows per thread
  constexpr int G = BLOCK / SPLIT;   // column groups per tile
  static_assert(KT % SPLIT == 0 && G % 32 == 0, "parts must be whole warps");
  __shared__ float xs[2][SPLIT][G * VEC];
  __shared__ double red[BLOCK / 32][R];
  const int tid = threadIdx.x, cg = tid % G, part = tid / G, r0 = part * R;
  float sacc[R];
#pragma unroll
  for (int m = 0; m < R; ++m) sacc[m] = 0.f;
  const float invK = 1.0f / (float)KR;
  const int64_t ntiles = (P + (int64_t)G * VEC - 1) / ((int64_t)G * VEC);
  int it = 0;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
    const int64_t col = (tile * G + cg) * VEC;
    const bool live = col < P;
    Pack<VEC> t[R];
    Pack<VEC> sum = p_zero<VEC>();
    if (live) {
#pragma unroll
      for (int m = 0; m < R; ++m) {
        if (!PAD || r0 + m < KR) t[m] = ld_stream<VEC>(theta + (size_t)(r0 + m) * ld + col);
        else t[m] = p_zero<VEC>();
      }
#pragma unroll
      for (int m = 0; m < R; ++m) sum = p_add<VEC>(sum, t[m]);
    }
    SCol<VEC>::st(xs[it & 1][part], cg, sum);
    __syncthreads();
    if (live) {
      Pack<VEC> mean = SCol<VEC>::ld(xs[it & 1][0], cg);
#pragma unroll
      for (int q = 1; q < SPLIT; ++q) mean = p_add<VEC>(mean, SCol<VEC>::ld(xs[it & 1][q], cg));
      mean = p_mul<VEC>(mean, invK);
#pragma unroll
      for (int m = 0; m < R; ++m) {
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
          const float d = t[m].v[i] - mean.v[i];
          sq = fmaf(d, d, sq);
        }
        sacc[m] += sq;
      }
    }
  }
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int m = 0; m < R; ++m) {
    double d = (double)sacc[m];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
    if (lane == 0) red[warp][m] = d;
  }
  __syncthreads();
  if (tid < KR) {                    // worker tid = rows of part tid / R, summed over that part's warps
    const int q = tid / R, j = tid % R;
    double d = 0.0;
#pragma unroll
    for (int w = 0; w < G / 32; ++w) d += red[q * (G / 32) + w][j];
    partials[(size_t)blockIdx.x * KR + tid] = d;
  }
  finalize_in_last_cta(partials, KR, out, done);
}

// Global average with many workers, same split: out = column mean as one row (out_is_vector) or
// written to every row.
template <int KT, int SPLIT, int VEC, int BLOCK>
__global__ void __launch_bounds__(BLOCK)
mix_mean_split_kernel(const float* __restrict__ in, float* __restrict__ out, int out_is_vector, int64_t P, int64_t ld) {
  constexpr int R = KT / SPLIT;
  constexpr int G = BLOCK / SPLIT;
  static_assert(KT % SPLIT == 0 && G % 32 == 0, "parts must be whole warps");
  __shared__ float xs[2][SPLIT][G * VEC];
  const int tid = threadIdx.x, cg = tid % G, part = tid / G, r0 = part * R;
  const float invK = 1.0f / (float)KT;
  const int64_t ntiles = (P + (int64_t)G * VEC - 1) / ((int64_t)G * VEC);
  int it = 0;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
    const int64_t col = (tile * G + cg) * VEC;
    const bool live = col < P;
    Pack<VEC> sum = p_zero<VEC>();
    if (live) {
      Pack<VEC> t[R];
#pragma unroll
      for (int m = 0; m < R; ++m) t[m] = ld_stream<VEC>(in + (size_t)(r0 + m) * ld + col);
#pragma unroll
      for (int m = 0; m < R; ++m) sum = p_add<VEC>(sum, t[m]);
    }
    SCol<VEC>::st(xs[it & 1][part], cg, sum);
    __syncthreads();
    if (live && (!out_is_vector || part == 0)) {
      Pack<VEC> mean = SCol<VEC>::ld(xs[it & 1][0], cg);
#pragma unroll
      for (int q = 1; q < SPLIT; ++q) mean = p_add<VEC>(mean, SCol<VEC>::ld(xs[it & 1][q], cg));
      mean = p_mul<VEC>(mean, invK);
      if (out_is_vector) {
        st_stream<VEC>(out + col, mean);
      } else {
#pragma unroll
        for (int m = 0; m < R; ++m) st_stream<VEC>(out + (size_t)(r0 + m) * ld + col, mean);
      }
    }
  }
}

// out[m] = sum_b partials[b][m], fixed order: one warp per worker, lanes stride the blocks,
// then a shuffle tree.  Deterministic.  The same sum as finalize_in_last_cta, as a launch of its
// own: used by the allocation-free entry point, which has no finished-CTA counter.
static __global__ void __launch_bounds__(32)
consensus_finalize_kernel(const double* __restrict__ partials, int nblocks, int K, double* __restrict__ out) {
  const int m = blockIdx.x, lane = threadIdx.x;
  double d = 0.0;
  for (int b = lane; b < nblocks; b += 32) d += partials[(size_t)b * K + m];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
  if (lane == 0) out[m] = d;
}

}  // namespace fgd
#endif
