// Stand-alone mix out = W in for 17 <= K <= 64 on the tensor cores: the tcgen05 3xTF32 contraction
// of the fused step (fgd_step_dense_tc.cuh: same W operand in shared memory, same split
//     W v ~= W_hi v_hi + W_hi v_lo + W_lo v_hi,  fp32 accumulators in tensor memory)
// with a data flow of its own.  A mix moves only 8 bytes per worker-parameter, so per tile the
// contraction, the tensor-memory round trip and the barrier hand-offs weigh much more than in the
// step; a kernel that holds its stage across them has one tile in flight per SM and is latency-bound.
// Here nothing waits on the arithmetic:
//   * the A operand v^T (M = 128 columns of the tile, K = workers) is read by the MMA from TENSOR
//     MEMORY: a consumer thread reads its H values of the staged box, splits them and writes v_hi /
//     v_lo into its own TMEM lane (lane = column) with tcgen05.st.  Shared memory is only the landing
//     zone of the TMA boxes -- a stage goes back to the producer as soon as the consumers hold it in
//     registers -- so the ring is deep (one 32 KB box per stage at K = 64: six stages in flight);
//   * operand buffers and accumulator are double-buffered in TMEM and a dedicated warp issues the
//     MMAs: the contraction of tile i runs while the consumers store the result of tile i - 1 and
//     read tile i + 1.
// Warps 0-7 consumers (thread (c, h): column c, workers [H h, H h + H)), warp 8 lane 0 TMA
// producer, warp 9 lane 0 MMA issuer (warp 9 owns the tensor-memory allocation).  Any mix is a
// dense matrix, so sparse mixes at these worker counts are densified by the caller and take this
// kernel too.  Every wait is bounded and gives up early once the CTA's abort flag is up; the
// producer waits for its copies, the MMA warp for its last commits, tensor memory is released.
#ifndef FGD_MIX_DENSE_TC_CUH_
#define FGD_MIX_DENSE_TC_CUH_

#include "fgd_step_dense_tc.cuh"

namespace fgd {

// tcgen05.mma with the A operand in tensor memory (lane = row of A, one 32-bit column per k).
__device__ __forceinline__ void umma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}

// Bounded wait that also gives up when the CTA's abort flag is up (looked at every 32 polls).
__device__ __forceinline__ bool mbar_wait_or_abort(uint32_t bar, uint32_t parity, uint32_t limit, const int* abort_flag) {
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
    if ((it & 31u) == 31u && *(const volatile int*)abort_flag) return false;
  }
  return false;
}

// The same with one polling lane per warp: the other lanes follow through the shuffle (32 times fewer
// polls on the barrier word; measured 2-4 % on the stand-alone mix).
__device__ __forceinline__ bool warp_wait_or_abort(uint32_t bar, uint32_t parity, uint32_t limit, const int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait_or_abort(bar, parity, limit, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

template <int KP>
struct TcMixShape {
  using S = TcShape<KP>;
  static constexpr int kCW = KP <= 32 ? 32 : 64;              // tensor-memory columns per buffer
  static constexpr int kTmemCols = KP <= 32 ? 256 : 512;      // 2 accumulators + 2 v_hi + 2 v_lo, a power of two
  static constexpr int kThreads = kTcConsumers + 64;          // consumers + producer warp + MMA warp
  // as many one-box stages as fit beside W_hi and W_lo (at most 8)
  static constexpr int kFit = (int)((227u * 1024u - 1024u - 128u - 2u * S::kWBytes) / S::kBox);
  static constexpr int kStages = kFit > 8 ? 8 : kFit;
  static constexpr size_t kSmem = 128 + (size_t)kStages * S::kBox + 2 * S::kWBytes;
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
__global__ void __launch_bounds__(TcMixShape<KP>::kThreads, 1)
mix_dense_tc_kernel(const TcMixArgs a, const DenseMix mx, const __grid_constant__ CUtensorMap tm_in) {
  using Shape = TcShape<KP>;
  constexpr int K = KP, T = kTcCols, H = Shape::kHalf, CONS = kTcConsumers, STAGES = TcMixShape<KP>::kStages;
  constexpr int CW = TcMixShape<KP>::kCW;
  constexpr uint32_t BOX = Shape::kBox, WB = Shape::kWBytes, SBO = Shape::kSbo;
  const int KR = FULL ? K : a.K;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  // full[STAGES], empty[STAGES], ready[2] (operands of buffer b stored), mma[2] (accumulator b complete)
  __shared__ __align__(8) unsigned long long bars[2 * STAGES + 4];
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_slot;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  unsigned char* wb_hi = base + (size_t)STAGES * BOX;
  unsigned char* wb_lo = wb_hi + WB;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[STAGES]);
  const uint32_t bar_ready = smem_u32(&bars[2 * STAGES]), bar_mma = smem_u32(&bars[2 * STAGES + 2]);
  const uint32_t spin = a.spin_limit;
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + T - 1) / T;
  const int64_t my_tiles = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, CONS / 32);     // one arrival per consumer warp
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_ready + 8u * b, CONS / 32);
      mbar_init(bar_mma + 8u * b, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < K * K; i += TcMixShape<KP>::kThreads) {   // B operand = W^T, K-major core matrices, zero-padded
    const int n = i / K, m = i % K;
    const float w = (FULL || (n < KR && m < KR)) ? mx.Wt[n * KR + m] : 0.f;
    const float hi = to_tf32(w);
    const uint32_t off = (uint32_t)(m >> 3) * SBO + (uint32_t)(n >> 2) * 128u + (uint32_t)(m & 7) * 16u + (uint32_t)(n & 3) * 4u;
    *reinterpret_cast<float*>(wb_hi + off) = hi;
    *reinterpret_cast<float*>(wb_lo + off) = w - hi;
  }
  if (warp == CONS / 32 + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)TcMixShape<KP>::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == CONS / 32) {
    // ===================================================== TMA producer (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait_or_abort(bar_empty + 8u * s, (use - 1) & 1, spin, &abort_flag);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = bar_full + 8u * s;
        mbar_expect_tx(full, BOX);
        if (i == a.skip_tile) continue;            // test hook: this load never arrives
        tma_load_2d(smem_u32(base + (size_t)s * BOX), &tm_in, (int)(tile * T), 0, full, policy);
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(a.status, FGD_ERR_TIMEOUT);
      }
      // never exit under a copy in flight: bounded wait for the last use of every stage
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)
        if (j != a.skip_tile) mbar_wait(bar_full + 8u * (uint32_t)(j % STAGES), (uint32_t)(j / STAGES) & 1, spin);
    }
  } else if (warp == CONS / 32 + 1) {
    // ===================================================== MMA issuer (one elected lane)
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B tf32, both K-major, N = K, M = 128
      constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(K >> 3) << 17) | ((uint32_t)(T >> 4) << 24);
      const uint32_t b_hi = smem_u32(wb_hi), b_lo = smem_u32(wb_lo);
      int64_t i = 0;
      for (; i < my_tiles; ++i) {
        const uint32_t b = (uint32_t)(i & 1);
        if (!mbar_wait_or_abort(bar_ready + 8u * b, (uint32_t)(i >> 1) & 1, spin, &abort_flag)) {
          *(volatile int*)&abort_flag = 1;
          atomicExch(a.status, FGD_ERR_TIMEOUT);
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_base + b * CW;
        const uint32_t a_hi = tmem_base + (2 + b) * CW, a_lo = tmem_base + (4 + b) * CW;
#pragma unroll
        for (int prod = 0; prod < 3; ++prod) {     // W_hi v_hi, W_hi v_lo, W_lo v_hi
          const uint32_t aa = prod == 1 ? a_lo : a_hi;
          const uint32_t bb = prod == 2 ? b_lo : b_hi;
#pragma unroll
          for (int ks = 0; ks < K / 8; ++ks) {
            const uint64_t db = umma_desc(bb + (uint32_t)ks * 256u, 128u, SBO, 0u);
            umma_tf32_ts(acc, aa + (uint32_t)ks * 8u, db, idesc, (prod | ks) ? 1u : 0u);
          }
        }
        umma_commit(bar_mma + 8u * b);
      }
      // tensor memory must not be released under a running MMA: wait (bounded) for the last commits
      for (int64_t j = (i > 2 ? i - 2 : 0); j < i; ++j)
        mbar_wait(bar_mma + 8u * (uint32_t)(j & 1), (uint32_t)(j >> 1) & 1, spin);
    }
  } else {
    // ===================================================== consumers: thread (c, h) = column c, workers [H h, H h + H)
    const int c = tid & (T - 1), h = tid >> 7, r0 = h * H;
    const int hr = FULL ? H : min(max(KR - r0, 0), H);
    const uint32_t t_acc = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)r0;   // + b * CW
    const uint32_t t_hi = t_acc + 2 * CW, t_lo = t_acc + 4 * CW;
    for (int64_t i = 0; i <= my_tiles; ++i) {
      if (i < my_tiles) {
        // ---------------- tile i: box -> registers -> split -> operand buffers i & 1
        const int s = (int)(i % STAGES);
        const uint32_t b = (uint32_t)(i & 1);
        const float* A = reinterpret_cast<const float*>(base + (size_t)s * BOX);
        if (!warp_wait_or_abort(bar_full + 8u * s, (uint32_t)(i / STAGES) & 1, spin, &abort_flag, lane)) {
          *(volatile int*)&abort_flag = 1;
          atomicExch(a.status, FGD_ERR_TIMEOUT);
          break;
        }
        float v[H];
#pragma unroll
        for (int n = 0; n < H; ++n) v[n] = A[(r0 + n) * T + c];
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8u * s);       // the box is in registers: refill the stage
#pragma unroll
        for (int n = 0; n < H; n += 8) {
          float hi[8], lo[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            hi[q] = to_tf32(v[n + q]);
            lo[q] = v[n + q] - hi[q];
          }
          tmem_st_8(t_hi + b * CW + (uint32_t)n, hi);
          tmem_st_8(t_lo + b * CW + (uint32_t)n, lo);
        }
        tmem_st_wait();
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_ready + 8u * b);
      }
      if (i > 0) {
        // ---------------- tile i - 1: accumulator -> HBM
        const int64_t j = i - 1;
        const uint32_t b = (uint32_t)(j & 1);
        const int64_t col = (blockIdx.x + j * (int64_t)gridDim.x) * T + c;
        if (!warp_wait_or_abort(bar_mma + 8u * b, (uint32_t)(j >> 1) & 1, spin, &abort_flag, lane)) {
          *(volatile int*)&abort_flag = 1;
          atomicExch(a.status, FGD_ERR_TIMEOUT);
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float r[H];
        tmem_ld_cols<H>(t_acc + b * CW, r);
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");   // ordered before what this thread signals next
        if (col < P) {
          float* const out_col = a.out + (size_t)r0 * ld + col;
#pragma unroll
          for (int m = 0; m < H; ++m) {
            if (FULL || m < hr) __stcs(out_col + (size_t)m * ld, r[m]);
          }
        }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == CONS / 32 + 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TcMixShape<KP>::kTmemCols) : "memory");
  }
}

}  // namespace fgd
#endif
