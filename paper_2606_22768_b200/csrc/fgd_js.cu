// JS functional-disagreement metric CD_JS (the paper's App. D.2) on logits resident in HBM.
//
// Per token position u: the top_k tokens of the parameter-averaged model's logits are selected
// (exact radix select, ties to the lower token index); every worker's distribution and the
// averaged model's are restricted to those tokens, renormalised, and compared with the
// normalised Jensen-Shannon distance sqrt(JS / ln 2), all in float64 in the log domain.
// Two kernels: one CTA per position selects the tokens, one warp per (worker, position) pair
// evaluates the distance; a third sums the distances of each worker in a fixed order.
#include <cuda_runtime.h>

#include <cstdio>

#include "fgd_internal.h"

using namespace fgd;

namespace {

constexpr int kSelBlock = 1024;
constexpr int kMaxTopK = 256;

int js_fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_thread_error, sizeof(g_thread_error), fmt, ap);
  va_end(ap);
  return status;
}

// fp32 -> unsigned key whose ASCENDING order is DESCENDING float order (largest logit first).
__device__ __forceinline__ uint32_t desc_key(float x) {
  const uint32_t b = __float_as_uint(x);
  const uint32_t asc = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  return ~asc;
}

// One CTA per row: indices of the k smallest keys (= k largest logits), ascending index order.
__global__ void __launch_bounds__(kSelBlock)
js_select_kernel(const float* __restrict__ avg_logits, int64_t V, int k, int32_t* __restrict__ idx_out) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining, s_less;
  __shared__ unsigned int warp_tot[2][kSelBlock / 32];
  __shared__ unsigned int s_eq_base, s_sel_base;
  const float* row = avg_logits + (size_t)blockIdx.x * V;
  int32_t* out = idx_out + (size_t)blockIdx.x * k;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_prefix = 0;
    s_remaining = (unsigned)k;
    s_less = 0;
  }
  // ---- radix select, 8 bits per pass from the top: key of the k-th smallest
  for (int pass = 3; pass >= 0; --pass) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const unsigned prefix = s_prefix;
    const unsigned hi_mask = pass == 3 ? 0u : (0xFFFFFFFFu << (8 * (pass + 1)));
#pragma unroll 4
    for (int64_t i = tid; i < V; i += kSelBlock) {
      const uint32_t key = desc_key(row[i]);
      if ((key & hi_mask) == (prefix & hi_mask)) atomicAdd(&hist[(key >> (8 * pass)) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned cum = 0, rem = s_remaining;
      int b = 0;
      for (; b < 256; ++b) {
        if (cum + hist[b] >= rem) break;
        cum += hist[b];
      }
      s_prefix = prefix | ((unsigned)b << (8 * pass));
      s_remaining = rem - cum;     // rank of the target inside bucket b
      s_less += cum;               // keys known to be smaller than the target
    }
    __syncthreads();
  }
  const unsigned target = s_prefix;
  const unsigned need_eq = (unsigned)k - s_less;   // how many keys equal to the target are taken
  if (tid == 0) {
    s_eq_base = 0;
    s_sel_base = 0;
  }
  __syncthreads();
  // ---- ordered compaction: selected = key < target, or key == target among the first need_eq
  for (int64_t base = 0; base < V; base += kSelBlock) {
    const int64_t i = base + tid;
    uint32_t key = 0xFFFFFFFFu;
    bool valid = i < V;
    if (valid) key = desc_key(row[i]);
    const bool is_eq = valid && key == target;
    // almost every chunk of a large vocabulary holds no candidate at all: one barrier and move on
    if (!__syncthreads_or(valid && key <= target)) continue;
    // block-wide exclusive scan of is_eq
    const unsigned eq_ballot = __ballot_sync(0xffffffffu, is_eq);
    if (lane == 0) warp_tot[0][warp] = __popc(eq_ballot);
    __syncthreads();
    unsigned eq_before = __popc(eq_ballot & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) eq_before += warp_tot[0][w];
    const unsigned eq_rank = s_eq_base + eq_before;
    const bool sel = valid && (key < target || (is_eq && eq_rank < need_eq));
    const unsigned sel_ballot = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) warp_tot[1][warp] = __popc(sel_ballot);
    __syncthreads();
    unsigned sel_before = __popc(sel_ballot & ((1u << lane) - 1u));
    unsigned eq_total = 0, sel_total = 0;
    for (int w = 0; w < kSelBlock / 32; ++w) {
      if (w < warp) sel_before += warp_tot[1][w];
      eq_total += warp_tot[0][w];
      sel_total += warp_tot[1][w];
    }
    if (sel) out[s_sel_base + sel_before] = (int32_t)i;
    __syncthreads();
    if (tid == 0) {
      s_eq_base += eq_total;
      s_sel_base += sel_total;
    }
    __syncthreads();
  }
}

__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {   // fixed butterfly: every lane gets the same bits
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// One warp per (worker m, position u): normalised JS distance over the selected tokens.
__global__ void __launch_bounds__(256)
js_distance_kernel(const float* __restrict__ worker_logits, const float* __restrict__ avg_logits,
                   const int32_t* __restrict__ idx, int K, int64_t U, int64_t V, int k, double* __restrict__ d_js) {
  const int64_t pair = (int64_t)blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (pair >= (int64_t)K * U) return;
  const int lane = threadIdx.x & 31;
  const int64_t m = pair / U, u = pair - m * U;
  const float* wrow = worker_logits + ((size_t)m * U + u) * V;
  const float* arow = avg_logits + (size_t)u * V;
  const int32_t* id = idx + (size_t)u * k;
  constexpr int PER = kMaxTopK / 32;
  double p[PER], q[PER];
  double pmax = -1e300, qmax = -1e300;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int t = lane + 32 * j;
    if (t < k) {
      const int32_t tok = id[t];
      p[j] = (double)wrow[tok];
      q[j] = (double)arow[tok];
      pmax = fmax(pmax, p[j]);
      qmax = fmax(qmax, q[j]);
    }
  }
  pmax = warp_max(pmax);
  qmax = warp_max(qmax);
  double ps = 0.0, qs = 0.0;
#pragma unroll
  for (int j = 0; j < PER; ++j)
    if (lane + 32 * j < k) {
      ps += exp(p[j] - pmax);
      qs += exp(q[j] - qmax);
    }
  const double plse = pmax + log(warp_sum(ps)), qlse = qmax + log(warp_sum(qs));
  const double ln_half = -0.69314718055994530942;
  double js = 0.0;
#pragma unroll
  for (int j = 0; j < PER; ++j)
    if (lane + 32 * j < k) {
      const double lp = p[j] - plse, lq = q[j] - qlse;
      const double hi = fmax(lp, lq), lo = fmin(lp, lq);
      const double lm = hi + log1p(exp(lo - hi)) + ln_half;      // log((p + q) / 2)
      js += 0.5 * exp(lp) * (lp - lm) + 0.5 * exp(lq) * (lq - lm);
    }
  js = warp_sum(js);
  if (lane == 0) d_js[pair] = sqrt(fmax(js, 0.0) / 0.69314718055994530942);
}

// cd_worker[m] = (1/U) sum_u d_js[m][u], one warp per worker, fixed order.
__global__ void __launch_bounds__(32)
js_mean_kernel(const double* __restrict__ d_js, int64_t U, double* __restrict__ cd_worker) {
  const int m = blockIdx.x, lane = threadIdx.x;
  double s = 0.0;
  for (int64_t u = lane; u < U; u += 32) s += d_js[(size_t)m * U + u];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xffffffffu, s, off);
  if (lane == 0) cd_worker[m] = s / (double)U;
}

}  // namespace

extern "C" int fgd_js_distance(int device, int K, int64_t U, int64_t V, int top_k, const float* worker_logits,
                               const float* avg_logits, int32_t* top_idx, double* d_js, double* cd_worker,
                               void* stream) {
  if (K < 1 || K > FGD_MAX_K || U < 1 || V < 1 || top_k < 1 || top_k > kMaxTopK || top_k > V)
    return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: need 1 <= K <= %d, U, V >= 1, 1 <= top_k <= min(%d, V)", FGD_MAX_K, kMaxTopK);
  if (U * (int64_t)K > 0x7fffffff * 8ll || U > 0x7fffffff)
    return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: too many positions");
  if (!worker_logits || !avg_logits || !top_idx || !d_js || !cd_worker) return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: NULL pointer");
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return js_fail(FGD_ERR_CUDA, "cudaGetDevice failed");
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return js_fail(FGD_ERR_CUDA, "cannot select device %d", device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  js_select_kernel<<<(unsigned)U, kSelBlock, 0, st>>>(avg_logits, V, top_k, top_idx);
  const int64_t pairs = (int64_t)K * U;
  js_distance_kernel<<<(unsigned)((pairs + 7) / 8), 256, 0, st>>>(worker_logits, avg_logits, top_idx, K, U, V, top_k, d_js);
  js_mean_kernel<<<K, 32, 0, st>>>(d_js, U, cd_worker);
  cudaError_t e = cudaGetLastError();
  if (prev != device) cudaSetDevice(prev);
  if (e != cudaSuccess) return js_fail(FGD_ERR_CUDA, "fgd_js_distance: launch failed: %s", cudaGetErrorString(e));
  return FGD_OK;
}
