// fgd_debug_stream_pattern: the fused outer step's HBM traffic without its arithmetic.
//
// A measurement aid (no counterpart in the paper).  The fused step reads theta_prev, theta_local and
// the momentum once and writes theta_new and the momentum once, in tiles of all K worker rows by a
// few hundred columns.  How fast HBM can serve exactly that access pattern -- 3 K row streams read and
// 2 K row streams written at the same time -- is what bounds the step, and it is measurably below
// what a plain two-stream copy reaches, the more so the more rows a tile has.  This kernel moves the
// same bytes in the same tiles through the same TMA stage ring and does nothing else: theta_new
// receives theta_prev's values and the momentum its own, so on an in-place call the tensors keep
// their contents.  Its time on the caller's own tensors is the step's access-pattern roofline.
#include <cuda.h>
#include <cuda_runtime.h>

#include "fgd_nvtx.h"
#include "fgd_tma_host.h"

using namespace fgd;

namespace {

constexpr int kProbeConsumers = 256;

struct ProbeArgs {
  float* theta_new;
  float* momentum;
  int64_t P, ld;
  int* status;
  uint32_t spin_limit;
};

// R rows x C columns per tile (R = K), STAGES stages of three such boxes.
template <int R, int C, int STAGES>
__global__ void __launch_bounds__(kProbeConsumers + 32, 1)
stream_pattern_kernel(const ProbeArgs a, const __grid_constant__ CUtensorMap tm_prev, const __grid_constant__ CUtensorMap tm_local,
                      const __grid_constant__ CUtensorMap tm_mom) {
  constexpr int BOXC = C < 256 ? C : 256, NBOX = C / BOXC;
  constexpr uint32_t TENS = R * C * 4, STAGE = 3 * TENS, BOX = R * BOXC * 4;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * STAGES];
  __shared__ int abort_flag;
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t ntiles = (a.P + C - 1) / C;
  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[STAGES + s]), kProbeConsumers / 32);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == kProbeConsumers / 32) {
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[STAGES + s]), (use - 1) & 1, a.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        const int64_t left = a.P - tile * C;
        const int nbox = left >= C ? NBOX : (int)((left + BOXC - 1) / BOXC);
        mbar_expect_tx(full, BOX * (uint32_t)(3 * nbox));
        const uint32_t dst = smem_u32(base + (size_t)s * STAGE);
        for (int b = 0; b < nbox; ++b) {
          const int c0 = (int)(tile * C + (int64_t)b * BOXC);
          tma_load_2d(dst + b * BOX, &tm_prev, c0, 0, full, policy);
          tma_load_2d(dst + TENS + b * BOX, &tm_local, c0, 0, full, policy);
          tma_load_2d(dst + 2 * TENS + b * BOX, &tm_mom, c0, 0, full, policy);
        }
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)     // never exit under a copy in flight
        mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, a.spin_limit);
    }
    return;
  }
  int64_t i = 0;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
    const int s = (int)(i % STAGES);
    if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars[s]), (uint32_t)(i / STAGES) & 1, a.spin_limit))) {
      *(volatile int*)&abort_flag = 1;
      atomicExch(a.status, FGD_ERR_TIMEOUT);
      break;
    }
    const float4* A = reinterpret_cast<const float4*>(base + (size_t)s * STAGE);
    const float4* B = A + TENS / 16;
    const float4* Cm = B + TENS / 16;
    constexpr int F4_PER_BOX = R * BOXC / 4, F4 = NBOX * F4_PER_BOX, PER = (F4 + kProbeConsumers - 1) / kProbeConsumers;
    float4 va[PER], vc[PER];
#pragma unroll
    for (int q = 0; q < PER; ++q) {
      const int e = q * kProbeConsumers + tid;
      if (e < F4) {
        va[q] = A[e];
        const float4 t = B[e];
        vc[q] = Cm[e];
        va[q].x += 0.f * t.x;                  // theta_local is read and kept alive; the value is unchanged (finite inputs)
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&bars[STAGES + s]));
#pragma unroll
    for (int q = 0; q < PER; ++q) {
      const int e = q * kProbeConsumers + tid;
      if (e < F4) {
        const int b = e / F4_PER_BOX, w = e % F4_PER_BOX, r = w / (BOXC / 4), c4 = w % (BOXC / 4);
        const int64_t col = tile * C + (int64_t)b * BOXC + 4 * c4;
        const size_t off = (size_t)r * a.ld + col;
        if (col + 3 < a.P) {
          __stcs(reinterpret_cast<float4*>(a.theta_new + off), va[q]);
          __stcs(reinterpret_cast<float4*>(a.momentum + off), vc[q]);
        } else {
          const float xa[4] = {va[q].x, va[q].y, va[q].z, va[q].w}, xc[4] = {vc[q].x, vc[q].y, vc[q].z, vc[q].w};
          for (int t = 0; t < 4; ++t)
            if (col + t < a.P) {
              a.theta_new[off + t] = xa[t];
              a.momentum[off + t] = xc[t];
            }
        }
      }
    }
  }
}

template <int R, int C, int STAGES>
int launch_probe(fgd_ctx* c, const float* theta_local, const float* theta_prev, float* momentum, float* theta_new, cudaStream_t st) {
  constexpr int BOXC = C < 256 ? C : 256;
  CUtensorMap tp, tl, tm;
  if (int rc = make_tensor_map(c, &tp, theta_prev, BOXC)) return rc;
  if (int rc = make_tensor_map(c, &tl, theta_local, BOXC)) return rc;
  if (int rc = make_tensor_map(c, &tm, momentum, BOXC)) return rc;
  const size_t smem = 128 + (size_t)STAGES * 3 * R * C * 4;
  const int64_t ntiles = (c->P + C - 1) / C;
  auto kern = stream_pattern_kernel<R, C, STAGES>;
  int grid = 0;
  if (int rc = persistent_grid(c, kern, kProbeConsumers + 32, smem, ntiles, &grid)) return rc;
  const ProbeArgs a{theta_new, momentum, c->P, c->ld, c->status, c->dbg_spin_limit ? c->dbg_spin_limit : kSpinLimit};
  kern<<<grid, kProbeConsumers + 32, smem, st>>>(a, tp, tl, tm);
  return check_launch(c, "stream_pattern_kernel");
}

}  // namespace

extern "C" int fgd_debug_stream_pattern(fgd_ctx* c, const float* theta_local, const float* theta_prev, float* momentum,
                                        float* theta_new, void* stream) {
  FGD_NVTX_RANGE("fgd_debug_stream_pattern");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_debug_stream_pattern: ctx is NULL");
  if (!theta_local || !theta_prev || !momentum || !theta_new) return fail(c, FGD_ERR_INVALID_ARG, "fgd_debug_stream_pattern: NULL tensor");
  if (!c->encode_tiled || c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096 || !aligned16(theta_local) || !aligned16(theta_prev) ||
      !aligned16(momentum) || !aligned16(theta_new))
    return fail(c, FGD_ERR_UNSUPPORTED, "fgd_debug_stream_pattern: needs 16-byte aligned tensors and ld %% 4 == 0");
  const Range r_new = mat_range(theta_new, c->K, c->P, c->ld), r_mom = mat_range(momentum, c->K, c->P, c->ld);
  const Range r_prev = mat_range(theta_prev, c->K, c->P, c->ld), r_loc = mat_range(theta_local, c->K, c->P, c->ld);
  if ((overlap(r_new, r_prev) && theta_new != theta_prev) || overlap(r_new, r_loc) || overlap(r_new, r_mom) ||
      overlap(r_mom, r_prev) || overlap(r_mom, r_loc))
    return fail(c, FGD_ERR_ALIAS, "fgd_debug_stream_pattern: forbidden overlap between tensors");
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  switch (c->K) {          // the tile shapes of the fused-step kernels at these worker counts (96 KB stages)
    case 4: return launch_probe<4, 1024, 4>(c, theta_local, theta_prev, momentum, theta_new, st);
    case 8: return launch_probe<8, 1024, 2>(c, theta_local, theta_prev, momentum, theta_new, st);
    case 16: return launch_probe<16, 512, 2>(c, theta_local, theta_prev, momentum, theta_new, st);
    case 32: return launch_probe<32, 256, 2>(c, theta_local, theta_prev, momentum, theta_new, st);
    case 64: return launch_probe<64, 128, 2>(c, theta_local, theta_prev, momentum, theta_new, st);
    default: return fail(c, FGD_ERR_UNSUPPORTED, "fgd_debug_stream_pattern: built for K = 4, 8, 16, 32, 64 (K = %d)", c->K);
  }
}
