// C-ABI entry points that touch the GPU: context, argument checks, kernel selection, launches.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <utility>

#include "fgd_ctx.h"
#include "fgd_kernels.cuh"
#include "fgd_nvtx.h"
#include "fgd_step_tma.h"

using namespace fgd;

extern "C" {

int fgd_create(fgd_ctx** out, int device, int K, int64_t P, int64_t ld) {
  FGD_NVTX_RANGE("fgd_create");
  if (!out) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_create: out is NULL");
  *out = nullptr;
  if (K < 1 || K > FGD_MAX_K) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_create: K=%d out of range [1, %d]", K, FGD_MAX_K);
  if (P < 1 || ld < P) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_create: need 1 <= P <= ld (P=%lld, ld=%lld)", (long long)P, (long long)ld);
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "cudaGetDeviceCount");
  if (device < 0 || device >= ndev) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_create: device %d of %d", device, ndev);
  DeviceGuard guard(device);
  if (!guard.ok) return fail(nullptr, FGD_ERR_CUDA, "fgd_create: cannot select device %d", device);
  fgd_ctx* c = new (std::nothrow) fgd_ctx();
  if (!c) return fail(nullptr, FGD_ERR_CUDA, "fgd_create: out of host memory");
  c->device = device;
  c->K = K;
  c->P = P;
  c->ld = ld;
  e = cudaDeviceGetAttribute(&c->num_sms, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
  if (e == cudaSuccess) e = cudaMalloc(&c->partials, sizeof(double) * (size_t)kMaxPartialBlocks * FGD_MAX_K);
  if (e == cudaSuccess) e = cudaMalloc(&c->status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->status, 0, sizeof(int));
  if (e == cudaSuccess) e = cudaMalloc(&c->done, sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(c->done, 0, sizeof(unsigned int));
  if (e == cudaSuccess) {
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      c->encode_tiled = nullptr;  // the TMA path is then unavailable; the register path still works
    cudaGetLastError();
  }
  if (e != cudaSuccess) {
    int rc = cuda_fail(nullptr, e, "fgd_create");
    delete c;
    return rc;
  }
  *out = c;
  return FGD_OK;
}

int fgd_destroy(fgd_ctx* c) {
  if (!c) return FGD_OK;
  DeviceGuard guard(c->device);
  cudaError_t e = cudaFree(c->partials);
  cudaFree(c->status);
  cudaFree(c->done);
  // resources of fgd_outer_step_from_host (all present or all null)
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->start_ev) cudaEventDestroy(c->start_ev);
  for (cudaEvent_t ev : c->chunk_ev)
    if (ev) cudaEventDestroy(ev);
  if (c->chunk_cd) cudaFree(c->chunk_cd);
  if (c->chunk_cd_host) cudaFreeHost(c->chunk_cd_host);
  delete c;
  return e == cudaSuccess ? FGD_OK : cuda_fail(nullptr, e, "fgd_destroy");
}

const char* fgd_last_error(const fgd_ctx* c) { return c ? c->err : g_thread_error; }

int fgd_set_path(fgd_ctx* c, int path) {
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_set_path: ctx is NULL");
  if (path < FGD_PATH_AUTO || path > FGD_PATH_TMA_FP32) return fail(c, FGD_ERR_INVALID_ARG, "fgd_set_path: unknown path %d", path);
  c->path = path;
  return FGD_OK;
}

int fgd_device_status(fgd_ctx* c, void* stream) {
  FGD_NVTX_RANGE("fgd_device_status");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_device_status: ctx is NULL");
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  int h = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FGD_CUDA(c, cudaMemcpyAsync(&h, c->status, sizeof(int), cudaMemcpyDeviceToHost, st));
  FGD_CUDA(c, cudaStreamSynchronize(st));
  if (h != 0) {
    FGD_CUDA(c, cudaMemsetAsync(c->status, 0, sizeof(int), st));
    return fail(c, h, "a device-side wait gave up (status %d); results of that launch are invalid", h);
  }
  return FGD_OK;
}
int64_t fgd_launch_count(const fgd_ctx* c) { return c ? c->launches : 0; }

int fgd_debug_set(fgd_ctx* c, int key, int64_t value) {
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_debug_set: ctx is NULL");
  switch (key) {
    case FGD_DEBUG_SPIN_LIMIT:
      if (value < 0 || value > (int64_t)0xffffffffu) return fail(c, FGD_ERR_INVALID_ARG, "fgd_debug_set: spin limit %lld out of range", (long long)value);
      c->dbg_spin_limit = (uint32_t)value;
      return FGD_OK;
    case FGD_DEBUG_SKIP_TILE:
      if (value < -1 || value > 0x7fffffff) return fail(c, FGD_ERR_INVALID_ARG, "fgd_debug_set: tile index %lld out of range", (long long)value);
      c->dbg_skip_tile = (int)value;
      return FGD_OK;
    case FGD_DEBUG_GOSSIP_PATH:
      if (value < 0 || value > 3) return fail(c, FGD_ERR_INVALID_ARG, "fgd_debug_set: gossip path %lld out of range", (long long)value);
      c->dbg_gossip_path = (int)value;
      return FGD_OK;
    default:
      return fail(c, FGD_ERR_INVALID_ARG, "fgd_debug_set: unknown key %d", key);
  }
}

int fgd_outer_grad(fgd_ctx* c, const float* theta_prev, const float* theta_local, float* g, void* stream) {
  FGD_NVTX_RANGE("fgd_outer_grad");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_outer_grad: ctx is NULL");
  if (!theta_prev || !theta_local || !g) return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_grad: NULL tensor");
  const Range rg = mat_range(g, c->K, c->P, c->ld);
  if (overlap(rg, mat_range(theta_prev, c->K, c->P, c->ld)) || overlap(rg, mat_range(theta_local, c->K, c->P, c->ld)))
    return fail(c, FGD_ERR_ALIAS, "fgd_outer_grad: g overlaps an input");
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int vec = pick_vec(4, c->P, c->ld, {theta_prev, theta_local, g});
  const int64_t total = (c->P / vec) * c->K;
  int64_t grid = (total + kGradBlock - 1) / kGradBlock;
  const int64_t cap = (int64_t)c->num_sms * 8;
  if (grid > cap) grid = cap;
  if (vec == 4) outer_grad_kernel<4, kGradBlock><<<(int)grid, kGradBlock, 0, st>>>(theta_prev, theta_local, g, c->K, c->P, c->ld);
  else if (vec == 2) outer_grad_kernel<2, kGradBlock><<<(int)grid, kGradBlock, 0, st>>>(theta_prev, theta_local, g, c->K, c->P, c->ld);
  else outer_grad_kernel<1, kGradBlock><<<(int)grid, kGradBlock, 0, st>>>(theta_prev, theta_local, g, c->K, c->P, c->ld);
  return check_launch(c, "outer_grad_kernel");
}

int fgd_mix(fgd_ctx* c, const fgd_mix_desc* desc, const float* in, float* out, int out_is_vector, void* stream) {
  FGD_NVTX_RANGE("fgd_mix");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_mix: ctx is NULL");
  if (!in || !out) return fail(c, FGD_ERR_INVALID_ARG, "fgd_mix: NULL tensor");
  if (int rc = validate_desc(desc, c->K, c->err, sizeof(c->err))) return rc;
  if (out_is_vector && desc->kind != FGD_MIX_MEAN)
    return fail(c, FGD_ERR_INVALID_ARG, "fgd_mix: a vector output needs FGD_MIX_MEAN");
  const Range rin = mat_range(in, c->K, c->P, c->ld);
  const Range rout = out_is_vector ? vec_range(out, c->P, sizeof(float)) : mat_range(out, c->K, c->P, c->ld);
  if (overlap(rin, rout) && (out_is_vector || out != in))
    return fail(c, FGD_ERR_ALIAS, "fgd_mix: out overlaps in (only out == in is allowed)");
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  const int K = c->K, KT = kt_of(K);
  const int vec = pick_vec(want_vec(KT), c->P, c->ld, {in, out});
  MixArgs a{in, out, c->P, c->ld, K, out_is_vector ? 1 : 0};
  const bool dense = desc->kind == FGD_MIX_DENSE;
  GatherMix gm;
  static thread_local DenseMix dm;
  if (dense) make_dense(desc, &dm);
  else if (int rc = make_gather(c, desc, &gm)) return rc;

  // global average with 32 / 64 workers: several threads share a column (see mix_mean_split_kernel)
  if (desc->kind == FGD_MIX_MEAN && (K == 32 || K == 64) && pick_vec(4, c->P, c->ld, {in, out}) == 4) {
    const int64_t cols = 4 * kSplitBlock / (K / 16);           // columns per tile: (block / SPLIT) groups of 4, SPLIT = K / 16
    const int64_t ntiles = (c->P + cols - 1) / cols;
    int grid = 0;
    auto launch = [&](auto kern) -> int {
      if (int rc = persistent_grid(c, kern, kSplitBlock, 0, ntiles, &grid)) return rc;
      kern<<<grid, kSplitBlock, 0, st>>>(in, out, out_is_vector ? 1 : 0, c->P, c->ld);
      return check_launch(c, "mix_mean_split_kernel");
    };
    return K == 64 ? launch(mix_mean_split_kernel<64, 4, 4, kSplitBlock>) : launch(mix_mean_split_kernel<32, 2, 4, kSplitBlock>);
  }

  // a sparse mix above 16 workers: the TMA-pipelined row gather, whatever the worker and slot counts
  // (5.4-5.9 TB/s; the tensor-core mix on the densified matrix: 2.2-5.6, the 32- / 64-worker column kernels: 5.3 / 4.1)
  if (!dense && !out_is_vector && gm.kind == KMIX_GATHER && K > 16 && c->path != FGD_PATH_REGISTER &&
      fgd_mix_gather_tma_eligible(c, in, out))
    return fgd_launch_mix_gather_tma(c, in, out, gm, st);

  // worker counts above 16 without a compile-time fp32 kernel, and dense matrices from K = 32 up:
  // the tensor-core kernel (any mix is a dense matrix, so a sparse or mean one is densified for it)
  // (not the global average: its load-and-add column kernel runs at 5.6-6.0 TB/s with any K, the densified one at 2.2-4.5)
  if (!out_is_vector && desc->kind != FGD_MIX_MEAN && (c->path == FGD_PATH_AUTO || c->path == FGD_PATH_TMA) &&
      fgd_mix_tc_eligible(c, in, dense)) {
    bool ok = true;
    if (!dense) {
      double Wd[FGD_MAX_K * FGD_MAX_K];
      ok = fgd_dense_matrix(desc, Wd) == FGD_OK;
      if (ok)
        for (int m = 0; m < K; ++m)
          for (int n = 0; n < K; ++n) dm.Wt[n * K + m] = (float)Wd[m * K + n];
    }
    if (ok) return fgd_launch_mix_dense_tc(c, in, out, dm, st);
  }

  // worker counts up to 16 that are not powers of two: compile-time kernels of their own (sparse and
  // mean mixes, four columns per thread; run-time K before: ring 3.7-4.3 TB/s, mean 4.3-5.9)
  if (!dense && small_odd_k(K) && pick_vec(4, c->P, c->ld, {in, out}) == 4) {
    return dispatch_small_k(K, [&]<int KTc>() -> int {
      const int64_t ntiles = (c->P + (int64_t)kBlock * 4 - 1) / ((int64_t)kBlock * 4);
      const size_t smem = desc->kind == FGD_MIX_MEAN ? 0 : sizeof(float) * (size_t)K * kBlock * 4;
      int grid = 0;
      auto launch = [&](auto kern) -> int {
        if (int rc = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return rc;
        kern<<<grid, kBlock, smem, st>>>(a, gm);
        return check_launch(c, "mix_kernel");
      };
      const int dt = (gm.kind == KMIX_GATHER && gm.D >= 1 && gm.D <= 4) ? (gm.D == 3 ? 4 : gm.D) : -1;
      if (dt == 1) return launch(mix_kernel<KTc, 4, false, kBlock, GatherMix, 1>);
      if (dt == 2) return launch(mix_kernel<KTc, 4, false, kBlock, GatherMix, 2>);
      if (dt == 4) return launch(mix_kernel<KTc, 4, false, kBlock, GatherMix, 4>);
      return launch(mix_kernel<KTc, 4, false, kBlock, GatherMix>);
    });
  }

  return dispatch_kv(KT, vec, [&]<int KTc, int VECc>() -> int {
    const int64_t ntiles = (c->P + (int64_t)kBlock * VECc - 1) / ((int64_t)kBlock * VECc);
    // the averaging path keeps everything in registers: no private columns, more CTAs per SM
    size_t smem = desc->kind == FGD_MIX_MEAN ? 0 : sizeof(float) * (size_t)K * kBlock * VECc;
    int grid = 0;
    if (dense) {
      smem += sizeof(float) * (size_t)K * K;
      auto kern = mix_kernel<KTc, VECc, true, kBlock, DenseMix>;
      if (int rc = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return rc;
      kern<<<grid, kBlock, smem, st>>>(a, dm);
    } else {
      auto launch = [&](auto kern) -> int {
        if (int rc = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return rc;
        kern<<<grid, kBlock, smem, st>>>(a, gm);
        return FGD_OK;
      };
      int rc = FGD_OK;
      // compile-time worker counts also get a compile-time neighbour count (fully unrolled gathers)
      // (three slots run as four, five to seven as eight -- K = 8 and 16 only: unused slots carry
      // weight 0 and point at the row itself)
      int dt = -1;
      if (KTc > 0 && gm.kind == KMIX_GATHER && gm.D >= 1)
        dt = gm.D <= 4 ? (gm.D == 3 ? 4 : gm.D) : ((KTc == 8 || KTc == 16) ? 8 : -1);
      if constexpr (KTc > 0) {
        if (dt == 1) rc = launch(mix_kernel<KTc, VECc, false, kBlock, GatherMix, 1>);
        else if (dt == 2) rc = launch(mix_kernel<KTc, VECc, false, kBlock, GatherMix, 2>);
        else if (dt == 4) rc = launch(mix_kernel<KTc, VECc, false, kBlock, GatherMix, 4>);
        else if (dt == 8) rc = launch(mix_kernel<(KTc == 8 || KTc == 16) ? KTc : 8, VECc, false, kBlock, GatherMix, 8>);
        else rc = launch(mix_kernel<KTc, VECc, false, kBlock, GatherMix>);
      } else {
        rc = launch(mix_kernel<KTc, VECc, false, kBlock, GatherMix>);
      }
      if (rc) return rc;
    }
    return check_launch(c, "mix_kernel");
  });
}

int fgd_outer_step(fgd_ctx* c, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused, const float* x,
                   int x_is_vector, const float* theta_local, const float* theta_prev, float* momentum,
                   float* theta_new, double lr, double mu, double* cd_sumsq, void* stream) {
  return fgd_outer_step_ex(c, mix2, mix1_fused, x, x_is_vector, theta_local, theta_prev, momentum, theta_new, lr, mu,
                           cd_sumsq, nullptr, stream);
}

// Worker counts up to 15 that are not powers of two have a register kernel compiled for that very count
// and a pipelined kernel that is either their own (3, 6, 12) or the next larger one run zero-padded (5 on 6,
// 7 on 8, 9-11 on 12, 13-15 on 16), which moves no extra HBM bytes but does the larger kernel's
// shared-memory traffic and arithmetic.  Which is faster was measured per structure (4 GB per tensor, in
// place, consensus sums on; TB/s register / pipelined):
//   9-11 workers: the register kernel everywhere (ring 5.96-6.00 / 4.7-5.5, dense 5.9 / 4.6-5.1, matrix x
//   5.7-6.2 / 5.0-5.5, ring + ring fused 6.1-6.4 / 4.6-5.3, matching fused 6.3-6.4 / 4.6-5.5);
//   6 and 12: their own pipelined kernel (6.0-6.6 / 5.4-6.3 the other way round);
//   dense Mix2: register at 3, 7, 13-15 (5.9-6.2 / 4.2-5.9), a tie at 5;
//   sparse Mix1 gathered in the kernel: register at 7 (6.0-6.4 / 4.8-5.7), at 5 from three neighbour slots
//   (6.3 / 5.5; ring 5.8 / 6.2), at 14 and 15 up to two slots (5.4-6.0 / 4.9-5.6; four slots 4.7-4.9 / 4.9-5.9),
//   pipelined at 3 and 13;
//   matrix-valued x: register up to 7 workers (6.2-6.5 / 5.7-6.5), pipelined at 13-15 (4.7-5.9 / 5.3-5.7);
//   x one value per column: register (5.9-6.3 / 5.2-5.9) except a light Mix2 at 7 (6.0 / 6.1-6.3).
static bool reg_beats_pipelined(int K, bool dense2, bool x_matrix, bool gossip1, int D2, int D1) {
  if (K == 6 || K == 12) return false;
  if (K >= 9 && K <= 11) return true;
  if (dense2) return K != 5;
  const int D = D1 > D2 ? D1 : D2;
  if (gossip1) {
    if (K == 7) return true;
    if (K == 5) return D >= 3;
    if (K >= 14) return D <= 2;
    return false;
  }
  if (x_matrix) return K <= 7;
  if (K == 7) return D2 >= 3;
  return true;
}

int fgd_outer_step_ex(fgd_ctx* c, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused, const float* x,
                      int x_is_vector, const float* theta_local, const float* theta_prev, float* momentum,
                      float* theta_new, double lr, double mu, double* cd_sumsq, const fgd_step_options* opts,
                      void* stream) {
  FGD_NVTX_RANGE("fgd_outer_step_ex");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_outer_step: ctx is NULL");
  if (!theta_local || !theta_prev || !momentum || !theta_new)
    return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step: NULL tensor");
  if (!(lr == lr) || !(mu == mu)) return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step: lr / mu is NaN");
  if (int rc = validate_desc(mix2, c->K, c->err, sizeof(c->err))) return rc;
  if (mix1_fused) {
    if (x) return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step: give either mix1_fused or x, not both");
    if (int rc = validate_desc(mix1_fused, c->K, c->err, sizeof(c->err))) return rc;
    if (mix1_fused->kind == FGD_MIX_DENSE)
      return fail(c, FGD_ERR_UNSUPPORTED,
                  "fgd_outer_step: a dense Mix1 is not fused; run fgd_mix first and pass its result as x");
  } else if (!x) {
    return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step: need mix1_fused or x");
  }
  const int K = c->K;
  const Range r_new = mat_range(theta_new, K, c->P, c->ld), r_mom = mat_range(momentum, K, c->P, c->ld);
  const Range r_prev = mat_range(theta_prev, K, c->P, c->ld), r_loc = mat_range(theta_local, K, c->P, c->ld);
  if (overlap(r_new, r_prev) && theta_new != theta_prev)
    return fail(c, FGD_ERR_ALIAS, "fgd_outer_step: theta_new partially overlaps theta_prev");
  if (overlap(r_new, r_loc) || overlap(r_new, r_mom) || overlap(r_mom, r_prev) || overlap(r_mom, r_loc))
    return fail(c, FGD_ERR_ALIAS, "fgd_outer_step: forbidden overlap between tensors");
  if (x) {
    const Range rx = x_is_vector ? vec_range(x, c->P, sizeof(float)) : mat_range(x, K, c->P, c->ld);
    if (overlap(rx, r_new) || overlap(rx, r_mom)) return fail(c, FGD_ERR_ALIAS, "fgd_outer_step: x overlaps an output");
  }
  if (cd_sumsq) {
    const Range rc_ = vec_range(cd_sumsq, K, sizeof(double));
    if (overlap(rc_, r_new) || overlap(rc_, r_mom) || overlap(rc_, r_prev) || overlap(rc_, r_loc))
      return fail(c, FGD_ERR_ALIAS, "fgd_outer_step: cd_sumsq overlaps a tensor");
  }
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  StepArgs a;
  a.theta_local = theta_local;
  a.theta_prev = theta_prev;
  a.momentum = momentum;
  a.theta_new = theta_new;
  a.x = x;
  a.partials = cd_sumsq ? c->partials : nullptr;
  a.cd_out = cd_sumsq;
  a.done = c->done;
  a.P = c->P;
  a.ld = c->ld;
  a.K = K;
  a.xsrc = mix1_fused ? XSRC_FUSED : (x_is_vector ? XSRC_VECTOR : XSRC_MATRIX);
  a.lr = (float)lr;
  a.mu = (float)mu;
  a.n_ranges = 0;
  a.avg_momentum = 0;
  a.x_next = nullptr;
  for (int i = 0; i < FGD_MAX_RANGES; ++i) a.range_lo[i] = a.range_hi[i] = 0;
  if (opts) {
    if (opts->n_ranges < 0 || opts->n_ranges > FGD_MAX_RANGES || (opts->n_ranges > 0 && !opts->mix2_ranges))
      return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step_ex: n_ranges=%d out of [0, %d] or ranges missing", opts->n_ranges, FGD_MAX_RANGES);
    for (int i = 0; i < opts->n_ranges; ++i) {
      const int64_t lo = opts->mix2_ranges[2 * i], hi = opts->mix2_ranges[2 * i + 1];
      if (lo < 0 || hi < lo || hi > c->P || lo % 4 != 0 || (hi % 4 != 0 && hi != c->P))
        return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step_ex: range %d = [%lld, %lld) must lie in [0, P] on multiples of 4 columns", i, (long long)lo, (long long)hi);
      a.range_lo[i] = lo;
      a.range_hi[i] = hi;
    }
    a.n_ranges = opts->n_ranges;
    if (opts->x_next) {
      const Range rn = vec_range(opts->x_next, c->P, sizeof(float));
      if (overlap(rn, r_new) || overlap(rn, r_mom) || overlap(rn, r_prev) || overlap(rn, r_loc) ||
          (x && overlap(rn, x_is_vector ? vec_range(x, c->P, sizeof(float)) : mat_range(x, K, c->P, c->ld))))
        return fail(c, FGD_ERR_ALIAS, "fgd_outer_step_ex: x_next overlaps another tensor");
      a.x_next = opts->x_next;
    }
    if (opts->average_momentum) {
      const bool mean1 = mix1_fused ? mix1_fused->kind == FGD_MIX_MEAN : (x_is_vector != 0);
      if (!mean1) return fail(c, FGD_ERR_UNSUPPORTED, "fgd_outer_step_ex: average_momentum needs Mix1 to be the global average");
      a.avg_momentum = 1;
    }
  }

  GatherMix g1, g2;
  memset(&g1, 0, sizeof(g1));
  g1.kind = KMIX_MEAN;
  if (mix1_fused)
    if (int rc = make_gather(c, mix1_fused, &g1)) return rc;
  a.stage_tp = (mix1_fused && g1.kind == KMIX_GATHER) ? 1 : 0;
  const bool dense2 = mix2->kind == FGD_MIX_DENSE;
  static thread_local DenseMix d2;
  if (dense2) make_dense(mix2, &d2);
  else if (int rc = make_gather(c, mix2, &g2)) return rc;

  const int KT = kt_of(K);
  int grid = 0;
  int rc = FGD_OK;
  FgdTmaShape shape{0, 0, 0};
  // Gather-heavy calls -- four or more neighbour slots in Mix2 together with a per-row x (a matrix,
  // or a gossip Mix1 gathered in the kernel) -- wait on shared-memory loads with eight consumer warps
  // (config 4: 88 % of the copy peak); sixteen warps of one column each hide that (96 %).  Every
  // lighter call measured better with eight warps of two columns (config 3: 98 % vs 97 %; a ring
  // Mix2 with a matrix-valued x: 93 % vs 92 %; a fused global average with four slots: 97 % vs 94 %).
  const bool heavy = !dense2 && g2.kind == KMIX_GATHER && g2.D >= 4 &&
                     (a.xsrc == XSRC_MATRIX || (a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER));
  const bool can_tma = fgd_tma_eligible(c, a, dense2, heavy, &shape);
  // Worker counts up to 64 without a compile-time fp32 kernel of their own: the tensor-core kernel
  // is the fastest fused step we have there, and any mix is also a dense matrix -- so a gather /
  // mean Mix2 is densified and takes it too.
  // K = 32 has a compile-time fp32 kernel that is the faster one for a light sparse Mix2 (at most two
  // neighbour slots) with x one value per column (ring: 5.8 TB/s against 5.6); with more slots
  // (hypercube: 2.4 TB/s against 5.6), a matrix-valued x (5.1 against 5.8) or a sparse Mix1 gathered
  // in the kernel (5.1 against 5.4) the tensor-core kernel wins.
  const bool tc_at_32 = dense2 || (g2.kind == KMIX_GATHER && g2.D > 2) || a.xsrc == XSRC_MATRIX ||
                        (a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER);
  bool can_tc = c->path != FGD_PATH_TMA_FP32 && fgd_tc_eligible(c, a, tc_at_32, g1);
  if (can_tc && !dense2) {
    double Wd[FGD_MAX_K * FGD_MAX_K];
    if (fgd_dense_matrix(mix2, Wd) != FGD_OK) can_tc = false;
    else
      for (int m = 0; m < K; ++m)
        for (int n = 0; n < K; ++n) d2.Wt[n * K + m] = (float)Wd[m * K + n];
  }
  const bool gossip1 = a.xsrc == XSRC_FUSED && g1.kind == KMIX_GATHER;
  const bool can_rows = K > 16 && fgd_step_rows_eligible(c, a, dense2, g2);
  // The row gather (fgd_step_rows.cu) takes a sparse Mix1 fused into the step and a matrix-valued x at 17-28 and
  // at 33-64 workers (TB/s rows / best other kernel; ring + ring fused K = 17 5.5/5.4, 21 5.9/4.6, 24 5.8/4.6,
  // 28 5.6/5.2, 33 5.7/3.7, 40 6.1/4.2, 48 6.2/4.7, 56 5.8/4.2, 64 5.7/4.8; matching fused 5.6-6.2/3.7-5.9; four slots
  // 4.6-5.4/3.2-4.7; ring Mix2 with a matrix x K = 17 6.3/4.3, 24 6.4/4.3, 33 5.5/4.3, 40 5.5/5.2, 56 6.1/4.5; between 58
  // and 60 workers it falls to 4.8 against 5.0-5.4 -- where its stages push the shared-memory carve-out to the
  // maximum and 28 KB of L1 are left for the 30 KB of x in flight one tile ahead, the likely cause -- so the
  // tensor-core kernel keeps a matrix x there).  Not
  // with five and more slots in BOTH mixes from 25 workers, where the tensor-core kernels (Mix2, from 49 workers
  // also Mix1, as MMAs whatever the slot count) are ahead (K = 64, six slots: 4.1/4.8); not at 29-32 workers, where
  // its one CTA per SM shows and the two-group tensor-core kernel wins (K = 31: 4.6/6.0).  x one value per column
  // stays where it was: the two are within 4 % of each other.
  const bool rows_auto = (gossip1 || (a.xsrc == XSRC_MATRIX && K <= 58)) && (K <= 28 || K >= 33) &&
                         !(gossip1 && K >= 25 && g1.D >= 5 && g2.D >= 5);
  if ((c->path == FGD_PATH_TMA && !can_tma && !can_tc) || (c->path == FGD_PATH_TMA_FP32 && !can_tma && !can_rows))
    return fail(c, FGD_ERR_UNSUPPORTED,
                "fgd_outer_step: the TMA path needs 16-byte aligned tensors, ld %% 4 == 0 and room for two stages");
  const bool reg_odd = small_odd_k(K) && pick_vec(4, c->P, c->ld, {theta_local, theta_prev, momentum, theta_new, x, a.x_next}) == 4;
  const bool reg_k = fgd_reg_k_built(K) && pick_vec(2, c->P, c->ld, {theta_local, theta_prev, momentum, theta_new, x, a.x_next}) == 2;
  // 17-31 workers: the register kernel compiled for that count against the tensor-core kernel zero-padded to
  // 32 (measured, TB/s register / tensor cores, K = 17 | 20 | 24 | 28): ring 6.0/5.2 | 6.0/5.9 | 5.6/5.7 | 5.7/5.6;
  // four slots 5.9/4.9 | 5.8/4.9 | 4.8/5.8 | 5.0/5.5; matrix x 4.3/3.1 | 4.3/3.6 | 3.5/4.3 | 3.4/5.0; ring + ring fused
  // 5.5/3.8 | 5.2/4.4 | 4.7/5.2 | 4.5/6.0; matching fused 6.2/3.8 | 5.7/4.3 | 5.4/5.1 | 5.0/5.9; dense 3.4/4.8 | 3.5/5.1.
  const int gslots = (gossip1 && !dense2) ? (g1.D > g2.D ? g1.D : g2.D) : 0;
  const bool reg_k_auto = reg_k && !dense2 && c->path == FGD_PATH_AUTO &&
                          (K <= 20 || (gossip1 && ((gslots <= 1 && K <= 25) || (gslots <= 2 && K <= 21))));
  const bool reg_odd_auto = reg_odd && reg_beats_pipelined(K, dense2, a.xsrc == XSRC_MATRIX, gossip1,
                                                           dense2 ? 0 : g2.D, gossip1 ? g1.D : 0);
  if (can_rows && (c->dbg_gossip_path == 3 ||
                   (c->dbg_gossip_path == 0 && ((c->path == FGD_PATH_TMA_FP32 && (!can_tma || KT == 0)) ||
                                                (c->path == FGD_PATH_AUTO && rows_auto))))) {
    rc = fgd_launch_step_rows(c, a, g2, g1, st, &grid);
  } else if (can_tc && c->path != FGD_PATH_REGISTER && !reg_k_auto) {
    rc = fgd_launch_step_dense_tc(c, a, d2, g1, st, &grid);
  } else if (can_tma && c->path != FGD_PATH_REGISTER && !reg_k_auto &&
             !(c->path == FGD_PATH_AUTO && (K <= 2 || (dense2 && (KT == 8 || KT == 16)) || reg_odd_auto))) {
    // (AUTO keeps the register kernel with one or two workers, where a tile is too little work per
    // pipeline hand-off, and for a dense Mix2 at K = 8 and 16, where its all-register W g product
    // measured 5.9 / 6.1 TB/s against 5.2 / 5.0 TB/s for the shared-memory version of the pipelined kernel)
    rc = fgd_launch_step_tma(c, a, dense2, g2, d2, g1, shape, st, &grid);
  } else if (reg_k) {
    rc = fgd_launch_step_reg_k(c, a, dense2, g2, d2, g1, st, &grid);
  } else if (reg_odd) {
    rc = dispatch_small_k(K, [&]<int KTc>() -> int {
      const int64_t ntiles = (c->P + (int64_t)kBlock * 4 - 1) / ((int64_t)kBlock * 4);
      const size_t col = sizeof(float) * (size_t)K * kBlock * 4;
      const size_t smem = col + (a.stage_tp ? col : 0) + (dense2 ? sizeof(float) * (size_t)K * K : 0);
      if (dense2) {
        auto kern = outer_step_kernel<KTc, 4, true, kBlock, DenseMix>;
        if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
        kern<<<grid, kBlock, smem, st>>>(a, d2, g1);
      } else {
        auto kern = outer_step_kernel<KTc, 4, false, kBlock, GatherMix>;
        if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
        kern<<<grid, kBlock, smem, st>>>(a, g2, g1);
      }
      return check_launch(c, "outer_step_kernel");
    });
  } else {
    const int vec = pick_vec(want_vec(KT), c->P, c->ld, {theta_local, theta_prev, momentum, theta_new, x, a.x_next});
    rc = dispatch_kv(KT, vec, [&]<int KTc, int VECc>() -> int {
      const int64_t ntiles = (c->P + (int64_t)kBlock * VECc - 1) / ((int64_t)kBlock * VECc);
      const size_t col = sizeof(float) * (size_t)K * kBlock * VECc;
      size_t smem = col + (a.stage_tp ? col : 0);
      if (dense2) {
        if (!StepTraits<KTc, VECc, true>::kRegArrays) smem += col + sizeof(float) * (size_t)K * kBlock;
        smem += sizeof(float) * (size_t)K * K;
        auto kern = outer_step_kernel<KTc, VECc, true, kBlock, DenseMix>;
        if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
        kern<<<grid, kBlock, smem, st>>>(a, d2, g1);
      } else {
        if (!StepTraits<KTc, VECc, false>::kRegArrays) smem += col + sizeof(float) * (size_t)K * kBlock;
        auto kern = outer_step_kernel<KTc, VECc, false, kBlock, GatherMix>;
        if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
        kern<<<grid, kBlock, smem, st>>>(a, g2, g1);
      }
      return check_launch(c, "outer_step_kernel");
    });
  }
  if (rc) return rc;
  return FGD_OK;   // (the consensus sums are finalised by the kernel's last CTA)
}

int fgd_consensus_distance(fgd_ctx* c, const float* theta, double* cd_sumsq, void* stream) {
  FGD_NVTX_RANGE("fgd_consensus_distance");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_consensus_distance: ctx is NULL");
  if (!theta || !cd_sumsq) return fail(c, FGD_ERR_INVALID_ARG, "fgd_consensus_distance: NULL pointer");
  if (overlap(vec_range(cd_sumsq, c->K, sizeof(double)), mat_range(theta, c->K, c->P, c->ld)))
    return fail(c, FGD_ERR_ALIAS, "fgd_consensus_distance: cd_sumsq overlaps theta");
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int K = c->K, KT = kt_of(K);
  const int vec = pick_vec(want_vec(KT), c->P, c->ld, {theta});
  int grid = 0;
  if ((K == 32 || K == 64) && pick_vec(4, c->P, c->ld, {theta}) == 4) {   // see consensus_split_kernel
    auto launch = [&](auto kern, int64_t ntiles) -> int {
      if (int r = persistent_grid(c, kern, kSplitBlock, 0, ntiles, &grid)) return r;
      kern<<<grid, kSplitBlock, 0, st>>>(theta, c->partials, c->P, c->ld, cd_sumsq, c->done, K);
      return check_launch(c, "consensus_split_kernel");
    };
    const int64_t cols = 4 * kSplitBlock / (K / 16);           // columns per tile
    const int64_t ntiles = (c->P + cols - 1) / cols;
    if (int r = K == 64 ? launch(consensus_split_kernel<64, 4, 4, kSplitBlock>, ntiles)
                        : launch(consensus_split_kernel<32, 2, 4, kSplitBlock>, ntiles))
      return r;
    return FGD_OK;
  }
  if (K > 16 && K < 64 && pick_vec(4, c->P, c->ld, {theta}) == 4) {        // 17-31 and 33-63 workers: zero-padded split kernels
    const int KP = K < 32 ? 32 : 64;                                       // (run-time K before: 1.3-3.7 TB/s)
    const int64_t cols = 4 * kSplitBlock / (KP / 16);
    const int64_t ntiles = (c->P + cols - 1) / cols;
    auto launch = [&](auto kern) -> int {
      if (int r = persistent_grid(c, kern, kSplitBlock, 0, ntiles, &grid)) return r;
      kern<<<grid, kSplitBlock, 0, st>>>(theta, c->partials, c->P, c->ld, cd_sumsq, c->done, K);
      return check_launch(c, "consensus_split_kernel");
    };
    return KP == 64 ? launch(consensus_split_kernel<64, 4, 4, kSplitBlock, true>)
                    : launch(consensus_split_kernel<32, 2, 4, kSplitBlock, true>);
  }
  if (small_odd_k(K) && pick_vec(4, c->P, c->ld, {theta}) == 4) {   // compile-time kernels for 3, 5-7, 9-15 workers
    return dispatch_small_k(K, [&]<int KTc>() -> int {
      const int64_t ntiles = (c->P + (int64_t)kBlock * 4 - 1) / ((int64_t)kBlock * 4);
      auto kern = consensus_kernel<KTc, 4, kBlock>;
      if (int r = persistent_grid(c, kern, kBlock, 0, ntiles, &grid)) return r;
      kern<<<grid, kBlock, 0, st>>>(theta, c->partials, K, c->P, c->ld, cd_sumsq, c->done);
      return check_launch(c, "consensus_kernel");
    });
  }
  int rc = dispatch_kv(KT, vec, [&]<int KTc, int VECc>() -> int {
    const int64_t ntiles = (c->P + (int64_t)kBlock * VECc - 1) / ((int64_t)kBlock * VECc);
    const size_t smem = KTc > 0 ? 0 : sizeof(float) * (size_t)K * kBlock * (VECc + 1);
    auto kern = consensus_kernel<KTc, VECc, kBlock>;
    if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
    kern<<<grid, kBlock, smem, st>>>(theta, c->partials, K, c->P, c->ld, cd_sumsq, c->done);
    return check_launch(c, "consensus_kernel");
  });
  return rc;
}

}  // extern "C"
