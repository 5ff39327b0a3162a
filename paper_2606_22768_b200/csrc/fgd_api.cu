// C-ABI entry points that touch the GPU: context, argument checks, kernel selection, launches.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <map>
#include <utility>

#include "fgd_kernels.cuh"
#include "fgd_step_tma.cuh"

using namespace fgd;

namespace {
constexpr int kBlock = 128;           // threads per CTA for the column kernels
constexpr int kGradBlock = 256;
constexpr int kMaxPartialBlocks = 148 * 16 * 2;
}  // namespace

struct fgd_ctx {
  int device = 0;
  int K = 0;
  int64_t P = 0, ld = 0;
  int num_sms = 0;
  double* partials = nullptr;  // [kMaxPartialBlocks][K]
  int* status = nullptr;       // device status word written by bounded waits that gave up
  int path = FGD_PATH_AUTO;    // which fused-step kernel family to use
  int max_smem_optin = 0;
  void* encode_tiled = nullptr;  // cuTensorMapEncodeTiled, resolved through the runtime
  int64_t launches = 0;
  char err[256] = "";
  std::map<std::pair<const void*, size_t>, int> occupancy;  // (kernel, smem) -> CTAs per SM
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
  if (smem > 48 * 1024)
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

int launch_finalize(fgd_ctx* c, int nblocks, double* out, cudaStream_t st) {
  consensus_finalize_kernel<<<c->K, 32, 0, st>>>(c->partials, nblocks, c->K, out);
  return check_launch(c, "consensus_finalize_kernel");
}


// ---- TMA-pipelined fused step ------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D map of a [K, ld] fp32 matrix restricted to its first P columns; box = boxc columns x K rows.
// Columns at or beyond P read as zero.
int make_tensor_map(fgd_ctx* c, CUtensorMap* map, const float* base, int boxc) {
  const cuuint64_t dims[2] = {(cuuint64_t)c->P, (cuuint64_t)c->K};
  const cuuint64_t strides[1] = {(cuuint64_t)c->ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)boxc, (cuuint32_t)c->K};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_tiled)(
      map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(c, FGD_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
  return FGD_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tile shapes of the TMA kernel.  A stage holds n_tensors x K x (consumers * vec) floats and at
// least two stages must fit in shared memory; measured on B200, 256 consumer threads with
// K * vec = 32 (a 96 KB stage, two stages) is the fastest shape, narrower tiles are the
// fall-back when the Mix1 result is a staged matrix (four tensors per stage).
struct TmaShape {
  int vec, consumers, stages;
};
const int kTmaShapes[][3] = {  // {KT, vec, consumers}, in order of preference per KT
    {0, 1, 128},
    {2, 4, 256}, {2, 4, 128},
    {4, 4, 256}, {4, 4, 128},
    {8, 4, 256}, {8, 4, 128},
    {16, 2, 256}, {16, 2, 128},
    {32, 1, 256}, {32, 1, 128},
    {64, 1, 128},
};

size_t tma_fixed_smem(int K, int KT, bool dense2, int consumers) {
  return 128 + (dense2 ? sizeof(float) * K * K : 0) + (KT == 0 ? sizeof(float) * K * consumers : 0);
}

// Can the TMA kernel run this call?  Picks the tile shape.
bool tma_eligible(const fgd_ctx* c, const StepArgs& a, bool dense2, TmaShape* out) {
  if (!c->encode_tiled) return false;
  if (c->ld % 4 != 0 || c->P >= (int64_t)0x7fffffff - 4096) return false;
  if (!aligned16(a.theta_prev) || !aligned16(a.theta_local) || !aligned16(a.momentum) || !aligned16(a.theta_new)) return false;
  if (a.xsrc == XSRC_MATRIX && !aligned16(a.x)) return false;
  const int K = c->K, KT = kt_of(K), NT = a.xsrc == XSRC_MATRIX ? 4 : 3;
  const size_t budget = (size_t)c->max_smem_optin - 4096;  // static shared memory + slack
  for (const auto& sh : kTmaShapes) {
    if (sh[0] != KT) continue;
    const int vec = sh[1], consumers = sh[2];
    if (a.xsrc == XSRC_VECTOR && (reinterpret_cast<uintptr_t>(a.x) % (sizeof(float) * vec)) != 0) continue;
    const size_t fixed = tma_fixed_smem(K, KT, dense2, consumers);
    const size_t stage = tma_stage_bytes(K, consumers * vec, NT);
    if (budget < fixed + 2 * stage) continue;
    int stages = (int)((budget - fixed) / stage);
    if (stages > kMaxStages) stages = kMaxStages;
    *out = {vec, consumers, stages};
    return true;
  }
  return false;
}

int launch_step_tma(fgd_ctx* c, const StepArgs& a, bool dense2, const GatherMix& g2, const DenseMix& d2,
                    const GatherMix& g1, TmaShape sh, cudaStream_t st, int* grid_out) {
  const int K = c->K, KT = kt_of(K);
  TmaStepArgs ta;
  ta.s = a;
  ta.status = c->status;
  ta.n_tensors = a.xsrc == XSRC_MATRIX ? 4 : 3;
  ta.stages = sh.stages;
  const int T = sh.consumers * sh.vec;
  const int boxc = T < 256 ? T : 256;
  CUtensorMap tp, tl, tm, tx;
  if (int rc = make_tensor_map(c, &tp, a.theta_prev, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tl, a.theta_local, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tm, a.momentum, boxc)) return rc;
  if (int rc = make_tensor_map(c, &tx, a.xsrc == XSRC_MATRIX ? a.x : a.theta_prev, boxc)) return rc;
  const size_t smem = tma_fixed_smem(K, KT, dense2, sh.consumers) + tma_stage_bytes(K, T, ta.n_tensors) * sh.stages;
  const int64_t ntiles = (c->P + T - 1) / T;
  auto go = [&]<int KTc, int VECc, int Cc>() -> int {
    int grid = 0;
    if (dense2) {
      auto kern = outer_step_tma_kernel<KTc, VECc, Cc, true, DenseMix>;
      if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
      kern<<<grid, Cc + 32, smem, st>>>(ta, d2, g1, tp, tl, tm, tx);
    } else {
      auto kern = outer_step_tma_kernel<KTc, VECc, Cc, false, GatherMix>;
      if (int r = persistent_grid(c, kern, Cc + 32, smem, ntiles, &grid)) return r;
      kern<<<grid, Cc + 32, smem, st>>>(ta, g2, g1, tp, tl, tm, tx);
    }
    *grid_out = grid;
    return check_launch(c, "outer_step_tma_kernel");
  };
#define FGD_TMA_CASE(kt, v, cc) \
  if (KT == kt && sh.vec == v && sh.consumers == cc) return go.template operator()<kt, v, cc>();
  FGD_TMA_CASE(0, 1, 128)
  FGD_TMA_CASE(2, 4, 256) FGD_TMA_CASE(2, 4, 128)
  FGD_TMA_CASE(4, 4, 256) FGD_TMA_CASE(4, 4, 128)
  FGD_TMA_CASE(8, 4, 256) FGD_TMA_CASE(8, 4, 128)
  FGD_TMA_CASE(16, 2, 256) FGD_TMA_CASE(16, 2, 128)
  FGD_TMA_CASE(32, 1, 256) FGD_TMA_CASE(32, 1, 128)
  FGD_TMA_CASE(64, 1, 128)
#undef FGD_TMA_CASE
  return fail(c, FGD_ERR_UNSUPPORTED, "internal: no TMA kernel for this shape");
}

}  // namespace

extern "C" {

int fgd_create(fgd_ctx** out, int device, int K, int64_t P, int64_t ld) {
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
  delete c;
  return e == cudaSuccess ? FGD_OK : cuda_fail(nullptr, e, "fgd_destroy");
}

const char* fgd_last_error(const fgd_ctx* c) { return c ? c->err : g_thread_error; }

int fgd_set_path(fgd_ctx* c, int path) {
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_set_path: ctx is NULL");
  if (path < FGD_PATH_AUTO || path > FGD_PATH_TMA) return fail(c, FGD_ERR_INVALID_ARG, "fgd_set_path: unknown path %d", path);
  c->path = path;
  return FGD_OK;
}

int fgd_device_status(fgd_ctx* c, void* stream) {
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

int fgd_outer_grad(fgd_ctx* c, const float* theta_prev, const float* theta_local, float* g, void* stream) {
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

  return dispatch_kv(KT, vec, [&]<int KTc, int VECc>() -> int {
    const int64_t ntiles = (c->P + (int64_t)kBlock * VECc - 1) / ((int64_t)kBlock * VECc);
    size_t smem = sizeof(float) * (size_t)K * kBlock * VECc;
    int grid = 0;
    if (dense) {
      smem += sizeof(float) * (size_t)K * K;
      auto kern = mix_kernel<KTc, VECc, true, kBlock, DenseMix>;
      if (int rc = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return rc;
      kern<<<grid, kBlock, smem, st>>>(a, dm);
    } else {
      auto kern = mix_kernel<KTc, VECc, false, kBlock, GatherMix>;
      if (int rc = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return rc;
      kern<<<grid, kBlock, smem, st>>>(a, gm);
    }
    return check_launch(c, "mix_kernel");
  });
}

int fgd_outer_step(fgd_ctx* c, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused, const float* x,
                   int x_is_vector, const float* theta_local, const float* theta_prev, float* momentum,
                   float* theta_new, double lr, double mu, double* cd_sumsq, void* stream) {
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
  a.P = c->P;
  a.ld = c->ld;
  a.K = K;
  a.xsrc = mix1_fused ? XSRC_FUSED : (x_is_vector ? XSRC_VECTOR : XSRC_MATRIX);
  a.lr = (float)lr;
  a.mu = (float)mu;

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
  TmaShape shape{0, 0, 0};
  const bool can_tma = tma_eligible(c, a, dense2, &shape);
  if (c->path == FGD_PATH_TMA && !can_tma)
    return fail(c, FGD_ERR_UNSUPPORTED,
                "fgd_outer_step: the TMA path needs 16-byte aligned tensors, ld %% 4 == 0 and room for two stages");
  if (can_tma && c->path != FGD_PATH_REGISTER) {
    rc = launch_step_tma(c, a, dense2, g2, d2, g1, shape, st, &grid);
  } else {
    const int vec = pick_vec(want_vec(KT), c->P, c->ld, {theta_local, theta_prev, momentum, theta_new, x});
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
  if (cd_sumsq) return launch_finalize(c, grid, cd_sumsq, st);
  return FGD_OK;
}

int fgd_consensus_distance(fgd_ctx* c, const float* theta, double* cd_sumsq, void* stream) {
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
  int rc = dispatch_kv(KT, vec, [&]<int KTc, int VECc>() -> int {
    const int64_t ntiles = (c->P + (int64_t)kBlock * VECc - 1) / ((int64_t)kBlock * VECc);
    const size_t smem = KTc > 0 ? 0 : sizeof(float) * (size_t)K * kBlock * (VECc + 1);
    auto kern = consensus_kernel<KTc, VECc, kBlock>;
    if (int r = persistent_grid(c, kern, kBlock, smem, ntiles, &grid)) return r;
    kern<<<grid, kBlock, smem, st>>>(theta, c->partials, K, c->P, c->ld);
    return check_launch(c, "consensus_kernel");
  });
  if (rc) return rc;
  return launch_finalize(c, grid, cd_sumsq, st);
}

}  // extern "C"
