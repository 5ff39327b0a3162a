// fgd_consensus_distance_noalloc: the consensus-distance reduction for callers that must not
// allocate.  Everything else in the library hangs its per-CTA partial sums on a context, and a
// context costs a cudaMalloc.  Some callers cannot pay that: code running inside a memory pool
// it does not own, a plug-in loaded into a process whose allocator is frozen after start-up,
// a monitoring hook that is invoked between two steps of somebody else's training loop and
// may not disturb the allocator state.  For them the partial sums live in a fixed array that
// is part of the library image itself.
//
// The array (kNoAllocBlocks x FGD_MAX_K doubles = 512 KiB) is resident on every GPU that loads
// the library, from load until the process exits.  It is shared by all calls: two calls that
// overlap on the same GPU (different streams, or different threads) race on it and give wrong
// sums, so callers must order them.  Nothing in it has to start at zero -- every slot a call
// reads is written earlier in that same call -- so no clearing is needed and stale contents
// from the previous call are harmless.
#include <cuda_runtime.h>

#include <cstdio>
#include <mutex>

#include "fgd_kernels.cuh"
#include "fgd_nvtx.h"

using namespace fgd;

namespace {

constexpr int kNoAllocBlocks = 1024;  // most CTAs a call may use = rows of the static scratch
constexpr int kNoAllocBlock = 128;    // threads per CTA
constexpr int kMaxDevices = 64;

// File-scope scratch.  In HOST code this name is only a handle for the runtime, not a device
// address: the kernels get the address cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) double g_noalloc_partials[kNoAllocBlocks * FGD_MAX_K];

struct DeviceSetup {
  bool done = false;
  double* scratch = nullptr;  // device address of g_noalloc_partials on this device
  int num_sms = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

int na_fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_thread_error, sizeof(g_thread_error), fmt, ap);
  va_end(ap);
  return status;
}

// One-time set-up for `device` (which must be current): resolve the scratch address and the SM
// count.  Neither call allocates.
int setup_device(int device, DeviceSetup** out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[device];
  if (!s.done) {
    double* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_partials);
    if (e != cudaSuccess || ptr == nullptr)
      return na_fail(FGD_ERR_CUDA, "cudaGetSymbolAddress(static scratch) failed on device %d: %s", device,
                     cudaGetErrorString(e));
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess || sms < 1)
      return na_fail(FGD_ERR_CUDA, "cannot read the SM count of device %d: %s", device, cudaGetErrorString(e));
    s.scratch = ptr;
    s.num_sms = sms;
    s.done = true;
  }
  *out = &s;
  return FGD_OK;
}

template <int KT, int VEC>
int launch_consensus(const float* theta, double* scratch, int K, int64_t P, int64_t ld, int grid, cudaStream_t st) {
  const size_t smem = KT > 0 ? 0 : sizeof(float) * (size_t)K * kNoAllocBlock * (VEC + 1);
  auto kern = consensus_kernel<KT, VEC, kNoAllocBlock>;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return na_fail(FGD_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
  }
  kern<<<grid, kNoAllocBlock, smem, st>>>(theta, scratch, K, P, ld, nullptr, nullptr);   // two-stage: finalised below
  return FGD_OK;
}

}  // namespace

extern "C" int fgd_consensus_distance_noalloc(int device, int K, int64_t P, int64_t ld, const float* theta,
                                              double* cd_sumsq, void* stream) {
  FGD_NVTX_RANGE("fgd_consensus_distance_noalloc");
  if (device < 0 || device >= kMaxDevices) return na_fail(FGD_ERR_INVALID_ARG, "device %d out of range", device);
  if (K < 1 || K > FGD_MAX_K)
    return na_fail(FGD_ERR_INVALID_ARG,
                   "K=%d exceeds the static scratch (%d CTAs x %d workers x 8 bytes); the limit is K <= %d", K,
                   kNoAllocBlocks, FGD_MAX_K, FGD_MAX_K);
  if (P < 1 || ld < P) return na_fail(FGD_ERR_INVALID_ARG, "need 1 <= P <= ld (P=%lld, ld=%lld)", (long long)P, (long long)ld);
  if (!theta || !cd_sumsq) return na_fail(FGD_ERR_INVALID_ARG, "NULL pointer");
  {  // the K output doubles must not lie inside the matrix they are computed from
    const uintptr_t t_lo = reinterpret_cast<uintptr_t>(theta);
    const uintptr_t t_hi = t_lo + (uintptr_t)(((int64_t)(K - 1) * ld + P) * (int64_t)sizeof(float));
    const uintptr_t o_lo = reinterpret_cast<uintptr_t>(cd_sumsq), o_hi = o_lo + (uintptr_t)K * sizeof(double);
    if (t_lo < o_hi && o_lo < t_hi) return na_fail(FGD_ERR_ALIAS, "cd_sumsq overlaps theta");
  }
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return na_fail(FGD_ERR_CUDA, "cudaGetDevice failed");
  if (prev != device && cudaSetDevice(device) != cudaSuccess)
    return na_fail(FGD_ERR_CUDA, "cannot select device %d", device);
  int rc = FGD_OK;
  DeviceSetup* s = nullptr;
  rc = setup_device(device, &s);
  if (rc == FGD_OK) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // same kernel selection as the context-based entry point, without its occupancy cache
    int KT = 0;
    switch (K) { case 2: case 4: case 8: case 16: case 32: case 64: KT = K; break; default: KT = 0; }
    int vec = KT == 0 ? 1 : (KT <= 16 ? 4 : (KT == 32 ? 2 : 1));
    while (vec > 1 && (P % vec != 0 || ld % vec != 0 || (reinterpret_cast<uintptr_t>(theta) % (sizeof(float) * vec)) != 0))
      vec >>= 1;
    const int64_t ntiles = (P + (int64_t)kNoAllocBlock * vec - 1) / ((int64_t)kNoAllocBlock * vec);
    int64_t grid = (int64_t)s->num_sms * 4;
    if (grid > ntiles) grid = ntiles;
    if (grid > kNoAllocBlocks) grid = kNoAllocBlocks;   // never more partial rows than the scratch holds
#define FGD_NA_CASE(kt, v) \
  else if (KT == kt && vec == v) rc = launch_consensus<kt, v>(theta, s->scratch, K, P, ld, (int)grid, st);
    if (false) {}
    FGD_NA_CASE(0, 1)
    FGD_NA_CASE(2, 4) FGD_NA_CASE(2, 2) FGD_NA_CASE(2, 1)
    FGD_NA_CASE(4, 4) FGD_NA_CASE(4, 2) FGD_NA_CASE(4, 1)
    FGD_NA_CASE(8, 4) FGD_NA_CASE(8, 2) FGD_NA_CASE(8, 1)
    FGD_NA_CASE(16, 4) FGD_NA_CASE(16, 2) FGD_NA_CASE(16, 1)
    FGD_NA_CASE(32, 2) FGD_NA_CASE(32, 1)
    FGD_NA_CASE(64, 1)
    else rc = na_fail(FGD_ERR_UNSUPPORTED, "internal: no kernel for K=%d vec=%d", K, vec);
#undef FGD_NA_CASE
    if (rc == FGD_OK) {
      consensus_finalize_kernel<<<K, 32, 0, st>>>(s->scratch, (int)grid, K, cd_sumsq);
      cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) rc = na_fail(FGD_ERR_CUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return rc;
}
