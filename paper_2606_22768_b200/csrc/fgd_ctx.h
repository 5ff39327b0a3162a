// Context structure and small host helpers shared by the translation units that launch kernels.
#ifndef FGD_CTX_H_
#define FGD_CTX_H_

#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <initializer_list>
#include <map>
#include <utility>

#include "fgd_internal.h"

using namespace fgd;  // internal header: only included by this library's own translation units

namespace {
constexpr int kBlock = 128;           // threads per CTA for the column kernels
constexpr int kSplitBlock = 256;      // threads per CTA for the kernels whose threads share a column (K = 32, 64)
constexpr int kGradBlock = 256;
constexpr int kMaxPartialBlocks = 148 * 16 * 2;
}  // namespace

struct fgd_ctx {
  int device = 0;
  int K = 0;
  int64_t P = 0, ld = 0;
  int num_sms = 0;
  double* partials = nullptr;  // [kMaxPartialBlocks][K]
  unsigned int* done = nullptr; // finished-CTA counter of the kernels that finalise the consensus sums themselves
  int* status = nullptr;       // device status word written by bounded waits that gave up
  int path = FGD_PATH_AUTO;    // which fused-step kernel family to use
  int max_smem_optin = 0;
  void* encode_tiled = nullptr;  // cuTensorMapEncodeTiled, resolved through the runtime
  int64_t launches = 0;
  uint32_t dbg_spin_limit = 0;   // fgd_debug_set: polls before a device-side wait gives up (0 = the default)
  int dbg_skip_tile = -1;        // fgd_debug_set: tile whose loads the pipelined kernels withhold (-1 = none)
  int dbg_gossip_path = 0;       // fgd_debug_set: 0 = measured choice, 1 = tensor-core gather, 2 = tensor-core MMAs, 3 = row-gather kernel
  char err[256] = "";
  std::map<std::pair<const void*, size_t>, int> occupancy;  // (kernel, smem) -> CTAs per SM
  // fgd_outer_step_from_host only (created by its first call): copy stream, one event per column
  // chunk, per-chunk consensus sums on the device and their pinned host copy
  bool streaming_ready = false;     // all of the below exist (set only after every one was created)
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t start_ev = nullptr;
  cudaEvent_t chunk_ev[FGD_MAX_CHUNKS] = {};
  double* chunk_cd = nullptr;       // device [FGD_MAX_CHUNKS][FGD_MAX_K]
  double* chunk_cd_host = nullptr;  // pinned host, same shape
};

namespace {

int fail(fgd_ctx* c, int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  if (c) vsnprintf(c->err, sizeof(c->err), fmt, ap);
  else vsnprintf(g_thread_error, sizeof(g_thread_error), fmt, ap);
  va_end(ap);
  return status;
}

int cuda_fail(fgd_ctx* c, cudaError_t e, const char* what) {
  return fail(c, FGD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define FGD_CUDA(c, call)                                   \
  do {                                                      \
    cudaError_t e_ = (call);                                \
    if (e_ != cudaSuccess) return cuda_fail(c, e_, #call);  \
  } while (0)

// Byte range a [K, ld] matrix with P used columns occupies.
struct Range {
  uintptr_t lo, hi;
};
Range mat_range(const void* p, int K, int64_t P, int64_t ld) {
  const uintptr_t b = reinterpret_cast<uintptr_t>(p);
  return {b, b + (uintptr_t)(((int64_t)(K - 1) * ld + P) * (int64_t)sizeof(float))};
}
Range vec_range(const void* p, int64_t n, size_t elt) {
  const uintptr_t b = reinterpret_cast<uintptr_t>(p);
  return {b, b + (uintptr_t)n * elt};
}
bool overlap(Range a, Range b) { return a.lo < b.hi && b.lo < a.hi; }

// Widest vector width usable for these pointers / sizes, capped at `want`.
int pick_vec(int want, int64_t P, int64_t ld, std::initializer_list<const void*> ptrs) {
  for (int v = want; v > 1; v >>= 1) {
    bool ok = (P % v == 0) && (ld % v == 0);
    for (const void* p : ptrs)
      if (p && (reinterpret_cast<uintptr_t>(p) % (sizeof(float) * v)) != 0) ok = false;
    if (ok) return v;
  }
  return 1;
}

// Kernel-side description of a non-dense mix (identity / mean / sparse).
int make_gather(fgd_ctx* c, const fgd_mix_desc* d, GatherMix* out) {
  const int K = d->K;
  memset(out, 0, sizeof(*out));
  if (d->kind == FGD_MIX_MEAN) {
    out->kind = KMIX_MEAN;
    return FGD_OK;
  }
  out->kind = KMIX_GATHER;
  for (int m = 0; m < K; ++m) {
    out->w_self[m] = 1.f;
    for (int j = 0; j < FGD_MAX_D; ++j) out->nbr[m * FGD_MAX_D + j] = m;
  }
  if (d->kind == FGD_MIX_IDENTITY) return FGD_OK;
  if (d->kind != FGD_MIX_SPARSE) return fail(c, FGD_ERR_INVALID_ARG, "internal: not a gather mix");
  double w_eff[FGD_MAX_K * FGD_MAX_D], ws_eff[FGD_MAX_K];
  effective_weights(d, w_eff, ws_eff);
  out->D = d->D;
  for (int m = 0; m < K; ++m) {
    out->w_self[m] = (float)ws_eff[m];
    for (int j = 0; j < d->D; ++j) {
      const int n = d->nbr[m * d->D + j];
      out->nbr[m * FGD_MAX_D + j] = n >= 0 ? n : m;
      out->w[m * FGD_MAX_D + j] = n >= 0 ? (float)w_eff[m * d->D + j] : 0.f;
    }
  }
  return FGD_OK;
}

void make_dense(const fgd_mix_desc* d, DenseMix* out) {
  const int K = d->K;
  for (int m = 0; m < K; ++m)
    for (int n = 0; n < K; ++n) out->Wt[n * K + m] = d->W[m * K + n];
}

// CTAs per SM for (kernel, block, smem); raises the dynamic shared-memory limit when needed.
template <typename Kern>
int ctas_per_sm(fgd_ctx* c, Kern kern, int block, size_t smem, int* out) {
  const auto key = std::make_pair(reinterpret_cast<const void*>(kern), smem);
  auto it = c->occupancy.find(key);
  if (it != c->occupancy.end()) {
    *out = it->second;
    return FGD_OK;
  }
  cudaFuncAttributes fa;
  FGD_CUDA(c, cudaFuncGetAttributes(&fa, kern));
  if (smem + fa.sharedSizeBytes > 48 * 1024)     // the 48 KB default covers static + dynamic shared memory
    FGD_CUDA(c, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int n = 0;
  FGD_CUDA(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, block, smem));
  if (n < 1) return fail(c, FGD_ERR_UNSUPPORTED, "kernel does not fit on an SM (smem %zu B)", smem);
  c->occupancy[key] = n;
  *out = n;
  return FGD_OK;
}

template <typename Kern>
int persistent_grid(fgd_ctx* c, Kern kern, int block, size_t smem, int64_t ntiles, int* grid) {
  int per_sm = 0;
  if (int rc = ctas_per_sm(c, kern, block, smem, &per_sm)) return rc;
  int64_t g = (int64_t)per_sm * c->num_sms;
  if (g > ntiles) g = ntiles;
  if (g > kMaxPartialBlocks) g = kMaxPartialBlocks;
  if (g < 1) g = 1;
  *grid = (int)g;
  return FGD_OK;
}

int check_launch(fgd_ctx* c, const char* what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(c, e, what);
  c->launches += 1;
  return FGD_OK;
}

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) ok = false;
    else if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

// ---- compile-time K / vector width selection -------------------------------------------
// KT = K for the instantiated worker counts, 0 (runtime-K generic kernel) otherwise.
int kt_of(int K) {
  switch (K) {
    case 2: case 4: case 8: case 16: case 32: case 64: return K;
    default: return 0;
  }
}
// The TMA-pipelined fused step is also instantiated for 3, 6 and 12 workers (clusters that are not
// a power of two); the stand-alone kernels and the register path run those with run-time K.
// The worker counts in between run zero-padded on the next of those kernels: 5 on 6, 7 on 8, 9-11 on
// 12, 13-15 on 16 (the padded rows never touch HBM).
int kt_tma_of(int K) {
  if (K == 3 || K == 6 || K == 12) return K;
  if (K == 5) return 6;
  if (K == 7) return 8;
  if (K >= 9 && K <= 11) return 12;
  if (K >= 13 && K <= 15) return 16;
  return kt_of(K);
}
int want_vec(int KT) { return KT == 0 ? 1 : (KT <= 16 ? 4 : (KT == 32 ? 2 : 1)); }

// Calls f.template operator()<KT, VEC>() for the (KT, VEC) pair chosen at run time.
template <typename F>
int dispatch_kv(int KT, int VEC, F&& f) {
#define FGD_CASE(kt, v) \
  if (KT == kt && VEC == v) return f.template operator()<kt, v>();
  FGD_CASE(0, 1)
  FGD_CASE(2, 4) FGD_CASE(2, 2) FGD_CASE(2, 1)
  FGD_CASE(4, 4) FGD_CASE(4, 2) FGD_CASE(4, 1)
  FGD_CASE(8, 4) FGD_CASE(8, 2) FGD_CASE(8, 1)
  FGD_CASE(16, 4) FGD_CASE(16, 2) FGD_CASE(16, 1)
  FGD_CASE(32, 2) FGD_CASE(32, 1)
  FGD_CASE(64, 1)
#undef FGD_CASE
  return FGD_ERR_UNSUPPORTED;
}

// The stand-alone mix and consensus kernels are also instantiated for the worker counts up to 16
// that are not powers of two (four columns per thread only): calls f.template operator()<KT>().
inline bool small_odd_k(int K) { return K >= 3 && K <= 15 && kt_of(K) == 0; }
template <typename F>
int dispatch_small_k(int K, F&& f) {
#define FGD_CASE(kt) \
  if (K == kt) return f.template operator()<kt>();
  FGD_CASE(3) FGD_CASE(5) FGD_CASE(6) FGD_CASE(7) FGD_CASE(9) FGD_CASE(10) FGD_CASE(11)
  FGD_CASE(12) FGD_CASE(13) FGD_CASE(14) FGD_CASE(15)
#undef FGD_CASE
  return FGD_ERR_UNSUPPORTED;
}

}  // namespace

#endif
