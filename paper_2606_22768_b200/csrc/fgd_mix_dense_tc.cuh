// Stand-alone mix out = W in for 17 <= K <= 64 on the tensor cores: the same tcgen05 3xTF32
// contraction, operand layout and TMA / mbarrier / TMEM choreography as the fused step in
// fgd_step_dense_tc.cuh, with one tensor per stage.  A stage holds the [KP x 128] box of `in`
// (overwritten in place by its tf32-rounded half, the A operand "hi") and a second buffer of the
// same size for the remainders ("lo").  Any mix is a dense matrix, so sparse mixes at these worker
// counts are densified by the caller and take this kernel too.
#ifndef FGD_MIX_DENSE_TC_CUH_
#define FGD_MIX_DENSE_TC_CUH_

#include "fgd_step_dense_tc.cuh"

namespace fgd {

template <int KP>
struct TcMixShape {
  using S = TcShape<KP>;
  static constexpr int kStages = KP <= 32 ? 4 : 3;
  // dynamic shared memory: alignment slack + stages x (box + lo buffer) + W_hi + W_lo
  static constexpr size_t kSmem = 128 + (size_t)kStages * 2 * S::kBox + 2 * S::kWBytes;
};

struct TcMixArgs {
  const float* in;   // only described by the tensor map; kept for symmetry with MixArgs
  float* out;
  int64_t P, ld;
  int K;
  int* status;
  uint32_t spin_limit;   // polls before a bounded wait gives up
  int skip_tile;         // test hook, see TmaStepArgs
};

template <int KP, bool FULL>
__global__ void __launch_bounds__(kTcConsumers + 32)
mix_dense_tc_kernel(const TcMixArgs a, const DenseMix mx, const __grid_constant__ CUtensorMap tm_in) {
  using Shape = TcShape<KP>;
  constexpr int K = KP, T = kTcCols, H = Shape::kHalf, CONS = kTcConsumers, STAGES = TcMixShape<KP>::kStages;
  constexpr uint32_t BOX = Shape::kBox, WB = Shape::kWBytes, SBO = Shape::kSbo;
  const int KR = FULL ? K : a.K;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * STAGES + 1];   // full[], empty[], mma
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  unsigned char* wb_hi = base + (size_t)STAGES * 2 * BOX;
  unsigned char* wb_lo = wb_hi + WB;
  const uint32_t mma_bar = smem_u32(&bars[2 * STAGES]);
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + T - 1) / T;

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[STAGES + s]), CONS);
    }
    mbar_init(mma_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < K * K; i += CONS + 32) {   // B operand = W^T, K-major core matrices, zero-padded
    const int n = i / K, m = i % K;
    const float w = (FULL || (n < KR && m < KR)) ? mx.Wt[n * KR + m] : 0.f;
    const float hi = to_tf32(w);
    const uint32_t off = (uint32_t)(m >> 3) * SBO + (uint32_t)(n >> 2) * 128u + (uint32_t)(m & 7) * 16u + (uint32_t)(n & 3) * 4u;
    *reinterpret_cast<float*>(wb_hi + off) = hi;
    *reinterpret_cast<float*>(wb_lo + off) = w - hi;
  }
  if (warp == CONS / 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)Shape::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == CONS / 32) {
    // ===================================================== producer (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[STAGES + s]), (use - 1) & 1, a.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        mbar_expect_tx(full, BOX);
        if (i == a.skip_tile) continue;            // test hook: this load never arrives
        tma_load_2d(smem_u32(base + (size_t)s * 2 * BOX), &tm_in, (int)(tile * T), 0, full, policy);
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      // never exit under a copy in flight: bounded wait for the last use of every stage
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)
        if (j != a.skip_tile) mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, a.spin_limit);
    }
  } else {
    // ===================================================== consumers: thread (c, h) = column c, workers [H h, H h + H)
    const int c = tid & (T - 1), h = tid >> 7, r0 = h * H;
    const int hr = FULL ? H : min(max(KR - r0, 0), H);
    const uint32_t op_row = (uint32_t)(c >> 3) * SBO + (uint32_t)(c & 7) * 16u;
    constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(K >> 3) << 17) | ((uint32_t)(T >> 4) << 24);
    int64_t i = 0;
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++i) {
      const int s = (int)(i % STAGES);
      const uint32_t use = (uint32_t)(i / STAGES);
      const int64_t col = tile * T + c;
      const bool live = col < P;
      unsigned char* stage = base + (size_t)s * 2 * BOX;
      float* A = reinterpret_cast<float*>(stage);          // in box -> hi operand
      unsigned char* L = stage + BOX;                      // lo operand
      float v[H];
      if (mbar_wait(smem_u32(&bars[s]), use & 1, a.spin_limit)) {
#pragma unroll
        for (int n = 0; n < H; ++n) v[n] = A[(r0 + n) * T + c];
      } else {
        *(volatile int*)&abort_flag = 1;
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      named_bar_sync(1, CONS);                    // every consumer has read its rows of the box
      if (*(volatile int*)&abort_flag) break;
#pragma unroll
      for (int n = 0; n < H; n += 4) {
        float4 hi, lo;
        hi.x = to_tf32(v[n]);     lo.x = v[n] - hi.x;
        hi.y = to_tf32(v[n + 1]); lo.y = v[n + 1] - hi.y;
        hi.z = to_tf32(v[n + 2]); lo.z = v[n + 2] - hi.z;
        hi.w = to_tf32(v[n + 3]); lo.w = v[n + 3] - hi.w;
        const uint32_t off = op_row + (uint32_t)((r0 + n) >> 2) * 128u;
        *reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(A) + off) = hi;
        *reinterpret_cast<float4*>(L + off) = lo;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      named_bar_sync(2, CONS);                    // operands complete; last tile's TMEM reads are done too
      if (tid == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_hi = smem_u32(A), a_lo = smem_u32(L);
        const uint32_t b_hi = smem_u32(wb_hi), b_lo = smem_u32(wb_lo);
#pragma unroll
        for (int prod = 0; prod < 3; ++prod) {     // W_hi in_hi, W_hi in_lo, W_lo in_hi
          const uint32_t aa = prod == 1 ? a_lo : a_hi;
          const uint32_t bb = prod == 2 ? b_lo : b_hi;
#pragma unroll
          for (int ks = 0; ks < K / 8; ++ks) {
            const uint64_t da = umma_desc(aa + (uint32_t)ks * 256u, 128u, SBO, 0u);
            const uint64_t db = umma_desc(bb + (uint32_t)ks * 256u, 128u, SBO, 0u);
            umma_tf32(tmem_base, da, db, idesc, (prod | ks) ? 1u : 0u);
          }
        }
        umma_commit(mma_bar);
      }
      if (!mbar_wait(mma_bar, (uint32_t)i & 1, a.spin_limit)) {
        *(volatile int*)&abort_flag = 1;          // seen by everyone at the next tile's barrier
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&bars[STAGES + s]));   // the MMA has consumed the operands: the stage can be refilled
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float r[H];
      tmem_ld_cols<H>(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)r0, r);
      if (live) {
        float* const out_col = a.out + (size_t)r0 * ld + col;
#pragma unroll
        for (int m = 0; m < H; ++m) {
          if (FULL || m < hr) __stcs(out_col + (size_t)m * ld, r[m]);
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == CONS / 32) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Shape::kTmemCols) : "memory");
  }
}

}  // namespace fgd
#endif
