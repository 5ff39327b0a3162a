// CUDA twin of the seeded input generator (see gen.py for the definition; same bits).
//
// Holds none of the method's arithmetic.  fgdin_fill writes fp32(scale_m * eps) (optionally
// added to what is already there); fgdin_local_steps is the stand-in for the H inner
// training steps between two outer rounds: theta_local = theta_prev + fp32(sigma_m * eps).
// It is deliberately integer-heavy (two 64-bit hashes per element), so it behaves like a
// compute kernel when it is overlapped with the side-stream Mix1.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

constexpr uint64_t kG = 0x9E3779B97F4A7C15ull;

__host__ __device__ inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

inline uint64_t row_key(uint64_t seed, uint64_t tensor_id, uint64_t rnd, uint64_t m) {
  uint64_t k = mix64(seed + kG);
  k = mix64((k ^ tensor_id) + kG);
  k = mix64((k ^ rnd) + kG);
  k = mix64((k ^ m) + kG);
  return k;
}

__device__ inline int sum16(uint64_t z) {
  const uint32_t lo = (uint32_t)z, hi = (uint32_t)(z >> 32);
  return (int)((lo & 0xFFFFu) + (lo >> 16) + (hi & 0xFFFFu) + (hi >> 16));
}

struct RowParams {
  uint64_t key[64];
  float scale[64];
};

// mode 0: out = scale*eps; mode 1: out = base + scale*eps (base may equal out)
__global__ void __launch_bounds__(256)
fill_kernel(float* out, const float* base, int K, int64_t P, int64_t ld, RowParams rp, int mode, float inv_std) {
  const int64_t total = (int64_t)K * P;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t m = i / P, p = i - m * P;
    const uint64_t za = mix64(rp.key[m] + (2 * (uint64_t)p + 1) * kG);
    const uint64_t zb = mix64(rp.key[m] + (2 * (uint64_t)p + 2) * kG);
    const int c = sum16(za) + sum16(zb) - 262140;
    const float eps = __fmul_rn((float)c, inv_std);
    const float d = __fmul_rn(rp.scale[m], eps);
    const size_t off = (size_t)m * ld + p;
    out[off] = mode ? __fadd_rn(base[off], d) : d;
  }
}

}  // namespace

extern "C" {

// out[m][p] (+)= fp32(scale[m] * eps(seed, tensor_id, rnd, m, p)).  shared_row != 0 uses
// worker index 0 for every row's key (one draw broadcast to all workers).
// scale: HOST [K].  inv_std: the fp32 constant from gen.py (passed in so both sides use the
// very same bits).  Returns 0 or the cudaError_t of the launch.
int fgdin_fill(float* out, const float* base, int K, int64_t P, int64_t ld, uint64_t seed, int tensor_id,
               int64_t rnd, const float* scale, int shared_row, int add_to_base, float inv_std, void* stream) {
  if (K < 1 || K > 64 || P < 1 || ld < P || !out || !scale || (add_to_base && !base)) return -1;
  RowParams rp;
  for (int m = 0; m < K; ++m) {
    rp.key[m] = row_key(seed, (uint64_t)tensor_id, (uint64_t)rnd, shared_row ? 0 : (uint64_t)m);
    rp.scale[m] = scale[m];
  }
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int64_t grid = ((int64_t)K * P + 255) / 256;
  if (grid > (int64_t)sms * 8) grid = (int64_t)sms * 8;
  fill_kernel<<<(int)grid, 256, 0, (cudaStream_t)stream>>>(out, base, K, P, ld, rp, add_to_base, inv_std);
  return (int)cudaGetLastError();
}

}  // extern "C"
