// Fused outer step with a sparse (gossip) Mix1 AND Mix2 both on the tensor cores, 17 <= K <= 64.
//
// The paper's LocalM1M2 configuration (App. A table: pairwise gossip for both mixes) and any other
// gossip Mix1 fused into the step need, per column, x = W1 theta_prev next to ghat = W2 g.  Gathering
// x row by row from the staged theta_prev box costs every consumer thread H (D + 1) run-time-indexed
// shared-memory loads per tile and keeps the stage busy meanwhile.  But Mix1 is a K x K contraction
// of the very box that is already staged, so here it is a second group of MMAs:
//     acc_g = W2 g,   acc_x = W1 theta_prev        (each 3 x TF32: W_hi a_hi + W_hi a_lo + W_lo a_hi)
// with BOTH A operands (g^T and theta_prev^T, M = 128 columns x K workers) handed to the MMA from
// TENSOR MEMORY: a consumer thread reads its rows of theta_prev, theta_local and the momentum out of
// the stage, forms g, splits g and theta_prev and writes the four operand blocks into its own TMEM
// lane with tcgen05.st; the epilogue reads ghat and x back from the two accumulators, eight rows at a
// time.  Shared memory only holds the TMA landing boxes and the two weight matrices (W2 from the dense
// descriptor, W1 assembled in shared memory from the sparse one), and a box goes back to the producer
// as soon as its values are in registers -- which is what lets a ring of single boxes (five 32 KB boxes
// beside 64 KB of weights at K = 64) keep enough bytes in flight.
// Warps 0-7 consumers (thread (c, h): column c, workers [H h, H h + H)), warp 8 lane 0 TMA producer,
// warp 9 lane 0 MMA issuer and owner of the tensor-memory allocation.  Tensor-memory columns, CW = 32
// or 64 each: acc_g, acc_x, g_hi, g_lo, t_hi, t_lo.  All waits are bounded and abortable; the producer
// waits for its copies, the MMA warp for its last commit, tensor memory is always released.
#ifndef FGD_STEP_GOSSIP_TC_CUH_
#define FGD_STEP_GOSSIP_TC_CUH_

#include "fgd_mix_dense_tc.cuh"

namespace fgd {

template <int KP>
struct TcGossipShape {
  using S = TcShape<KP>;
  static constexpr int kCW = KP <= 32 ? 32 : 64;
  static constexpr int kTmemCols = KP <= 32 ? 256 : 512;        // 6 CW rounded up to a power of two
  static constexpr int kThreads = kTcConsumers + 64;
  // ring of single boxes beside W2_hi, W2_lo, W1_hi, W1_lo; a tile takes three boxes
  static constexpr int kFit = (int)((227u * 1024u - 2048u - 128u - 4u * S::kWBytes) / S::kBox);
  static constexpr int kBoxes = kFit > 12 ? 12 : kFit;
  static_assert(kBoxes >= 4, "the ring must hold more than one tile");
  static constexpr size_t kSmem = 128 + (size_t)kBoxes * S::kBox + 4 * S::kWBytes;
};

template <int KP, bool FULL>
__global__ void __launch_bounds__(TcGossipShape<KP>::kThreads, 1)
outer_step_gossip_tc_kernel(const TmaStepArgs ta, const DenseMix m2, const GatherMix m1,
                            const __grid_constant__ CUtensorMap tm_prev, const __grid_constant__ CUtensorMap tm_local,
                            const __grid_constant__ CUtensorMap tm_mom) {
  using Shape = TcShape<KP>;
  constexpr int K = KP, T = kTcCols, H = Shape::kHalf, CONS = kTcConsumers, NB = TcGossipShape<KP>::kBoxes;
  constexpr int CW = TcGossipShape<KP>::kCW;
  constexpr uint32_t BOX = Shape::kBox, WB = Shape::kWBytes, SBO = Shape::kSbo;
  const int KR = FULL ? K : ta.s.K;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * NB + 2];   // full[NB], empty[NB], ready, mma
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_slot;
  __shared__ float xchg[2][T];      // the two halves of a column exchange their theta_new sums

  const StepArgs& a = ta.s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool want_cd = a.partials != nullptr;
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
  unsigned char* w2_hi = base + (size_t)NB * BOX;
  unsigned char* w2_lo = w2_hi + WB;
  unsigned char* w1_hi = w2_lo + WB;
  unsigned char* w1_lo = w1_hi + WB;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[NB]);
  const uint32_t bar_ready = smem_u32(&bars[2 * NB]), bar_mma = smem_u32(&bars[2 * NB + 1]);
  const uint32_t spin = ta.spin_limit;
  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + T - 1) / T;
  const int64_t my_tiles = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  // operand layout of a weight matrix: element (m, n) of W^T as an N x K (m x n) K-major matrix
  auto w_off = [](int m, int n) {
    return (uint32_t)(m >> 3) * SBO + (uint32_t)(n >> 2) * 128u + (uint32_t)(m & 7) * 16u + (uint32_t)(n & 3) * 4u;
  };

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < NB; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, CONS / 32);      // one arrival per consumer warp
    }
    mbar_init(bar_ready, 1);
    mbar_init(bar_mma, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // W2 from the dense descriptor (zero-padded); W1 starts as zeros ...
  for (int i = tid; i < K * K; i += TcGossipShape<KP>::kThreads) {
    const int n = i / K, m = i % K;
    const float w = (FULL || (n < KR && m < KR)) ? m2.Wt[n * KR + m] : 0.f;
    const float hi = to_tf32(w);
    const uint32_t off = w_off(m, n);
    *reinterpret_cast<float*>(w2_hi + off) = hi;
    *reinterpret_cast<float*>(w2_lo + off) = w - hi;
    *reinterpret_cast<float*>(w1_hi + off) = 0.f;
    *reinterpret_cast<float*>(w1_lo + off) = 0.f;
  }
  __syncthreads();
  // ... and receives the sparse description: self weight on the diagonal, one entry per neighbour slot
  // (a row has no duplicate neighbours; unused slots carry weight 0 and are skipped)
  for (int i = tid; i < KR * (FGD_MAX_D + 1); i += TcGossipShape<KP>::kThreads) {
    const int m = i / (FGD_MAX_D + 1), j = i % (FGD_MAX_D + 1);
    float w;
    int n;
    if (j == FGD_MAX_D) { w = m1.w_self[m]; n = m; }
    else { w = j < m1.D ? m1.w[m * FGD_MAX_D + j] : 0.f; n = m1.nbr[m * FGD_MAX_D + j]; }
    if (w != 0.f && (j == FGD_MAX_D || n != m)) {
      const float hi = to_tf32(w);
      const uint32_t off = w_off(m, n);
      *reinterpret_cast<float*>(w1_hi + off) = hi;
      *reinterpret_cast<float*>(w1_lo + off) = w - hi;
    }
  }
  if (warp == CONS / 32 + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)TcGossipShape<KP>::kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;

  float sacc[H];
#pragma unroll
  for (int m = 0; m < H; ++m) sacc[m] = 0.f;

  if (warp == CONS / 32) {
    // ===================================================== TMA producer (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t g = 0;                                  // boxes issued: three per tile (theta_prev, theta_local, momentum)
      bool ok = true;
      for (int64_t i = 0; i < my_tiles && ok; ++i) {
        const int c0 = (int)((blockIdx.x + i * (int64_t)gridDim.x) * T);
        for (int t = 0; t < 3; ++t, ++g) {
          const int s = (int)(g % NB);
          const uint32_t use = (uint32_t)(g / NB);
          if (use > 0) ok = mbar_wait_or_abort(bar_empty + 8u * s, (use - 1) & 1, spin, &abort_flag);
          if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
          mbar_expect_tx(bar_full + 8u * s, BOX);
          if (i == ta.skip_tile) continue;            // test hook: these loads never arrive
          tma_load_2d(smem_u32(base + (size_t)s * BOX), t == 0 ? &tm_prev : (t == 1 ? &tm_local : &tm_mom), c0, 0,
                      bar_full + 8u * s, policy);
        }
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      // never exit under a copy in flight: bounded wait for the last use of every box
      for (int64_t j = (g > NB ? g - NB : 0); j < g; ++j)
        if (j / 3 != ta.skip_tile) mbar_wait(bar_full + 8u * (uint32_t)(j % NB), (uint32_t)(j / NB) & 1, spin);
    }
  } else if (warp == CONS / 32 + 1) {
    // ===================================================== MMA issuer (one elected lane)
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(K >> 3) << 17) | ((uint32_t)(T >> 4) << 24);
      const uint32_t bw[2][2] = {{smem_u32(w2_hi), smem_u32(w2_lo)}, {smem_u32(w1_hi), smem_u32(w1_lo)}};
      int64_t i = 0;
      for (; i < my_tiles; ++i) {
        if (!mbar_wait_or_abort(bar_ready, (uint32_t)i & 1, spin, &abort_flag)) {
          *(volatile int*)&abort_flag = 1;
          atomicExch(ta.status, FGD_ERR_TIMEOUT);
          break;
        }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int which = 0; which < 2; ++which) {      // 0: acc_g = W2 g, 1: acc_x = W1 theta_prev
          const uint32_t acc = tmem_base + (uint32_t)which * CW;
          const uint32_t a_hi = tmem_base + (uint32_t)(2 + 2 * which) * CW, a_lo = a_hi + CW;
#pragma unroll
          for (int prod = 0; prod < 3; ++prod) {       // W_hi a_hi, W_hi a_lo, W_lo a_hi
            const uint32_t aa = prod == 1 ? a_lo : a_hi;
            const uint32_t bb = bw[which][prod == 2 ? 1 : 0];
#pragma unroll
            for (int ks = 0; ks < K / 8; ++ks) {
              const uint64_t db = umma_desc(bb + (uint32_t)ks * 256u, 128u, SBO, 0u);
              umma_tf32_ts(acc, aa + (uint32_t)ks * 8u, db, idesc, (prod | ks) ? 1u : 0u);
            }
          }
        }
        umma_commit(bar_mma);
      }
      if (i > 0) mbar_wait(bar_mma, (uint32_t)(i - 1) & 1, spin);   // never release tensor memory under a running MMA
    }
  } else {
    // ===================================================== consumers
    const int c = tid & (T - 1), h = tid >> 7, r0 = h * H;
    const uint32_t t_lane = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)r0;
    const uint32_t t_accg = t_lane, t_accx = t_lane + CW, t_ghi = t_lane + 2 * CW, t_glo = t_lane + 3 * CW;
    const uint32_t t_thi = t_lane + 4 * CW, t_tlo = t_lane + 5 * CW;
    const float invK = 1.0f / (float)KR;
    const int hr = FULL ? H : min(max(KR - r0, 0), H);
    const float lr = a.lr, mu = a.mu;
    for (int64_t i = 0; i < my_tiles; ++i) {
      const int64_t col = (blockIdx.x + i * (int64_t)gridDim.x) * T + c;
      const bool live = col < P;
      // ---- the tile's three boxes -> registers; the boxes go back at once
      const int64_t g0 = 3 * i;
      bool got = true;
#pragma unroll
      for (int t = 0; t < 3; ++t)
        got = got && warp_wait_or_abort(bar_full + 8u * (uint32_t)((g0 + t) % NB), (uint32_t)((g0 + t) / NB) & 1, spin, &abort_flag, lane);
      float v[H];
      if (got) {
        const float* A = reinterpret_cast<const float*>(base + (size_t)((g0 + 0) % NB) * BOX);   // theta_prev
        const float* B = reinterpret_cast<const float*>(base + (size_t)((g0 + 1) % NB) * BOX);   // theta_local
        const float* C = reinterpret_cast<const float*>(base + (size_t)((g0 + 2) % NB) * BOX);   // momentum
#pragma unroll
        for (int n = 0; n < H; n += 8) {
          float thi[8], tlo[8], ghi[8], glo[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float tp = A[(r0 + n + q) * T + c];
            const float g = tp - B[(r0 + n + q) * T + c];
            thi[q] = to_tf32(tp);
            tlo[q] = tp - thi[q];
            ghi[q] = to_tf32(g);
            glo[q] = g - ghi[q];
          }
          tmem_st_8(t_thi + (uint32_t)n, thi);
          tmem_st_8(t_tlo + (uint32_t)n, tlo);
          tmem_st_8(t_ghi + (uint32_t)n, ghi);
          tmem_st_8(t_glo + (uint32_t)n, glo);
        }
#pragma unroll
        for (int m = 0; m < H; ++m) v[m] = C[(r0 + m) * T + c];
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
#pragma unroll
          for (int t = 0; t < 3; ++t) mbar_arrive(bar_empty + 8u * (uint32_t)((g0 + t) % NB));
        }
        tmem_st_wait();
      } else {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      named_bar_sync(1, CONS);                    // every operand of the tile is in tensor memory
      if (*(volatile int*)&abort_flag) break;     // uniform: raised before the barrier
      if (tid == 0) mbar_arrive(bar_ready);
      const bool done = warp_wait_or_abort(bar_mma, (uint32_t)i & 1, spin, &abort_flag, lane);
      if (!done) {
        *(volatile int*)&abort_flag = 1;          // seen by everyone at the barrier below
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // ---- epilogue: ghat and x come back eight rows at a time (double-buffered)
      float asum = 0.f;
      float* const mom_col = a.momentum + (size_t)r0 * ld + col;
      float* const new_col = a.theta_new + (size_t)r0 * ld + col;
      float gh8[2][8], x8[2][8];
      tmem_ld_8(t_accg, gh8[0]);
      tmem_ld_8(t_accx, x8[0]);
#pragma unroll
      for (int mb = 0; mb < H; mb += 8) {
        const int cur = (mb / 8) & 1;
        tmem_ld_wait();
        if (mb + 8 < H) {
          tmem_ld_8(t_accg + (uint32_t)(mb + 8), gh8[cur ^ 1]);
          tmem_ld_8(t_accx + (uint32_t)(mb + 8), x8[cur ^ 1]);
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int m = mb + q;
          const bool row_live = FULL || m < hr;
          const float vn = fmaf(mu, v[m], gh8[cur][q]);
          const float tn = fmaf(-lr, fmaf(mu, vn, gh8[cur][q]), x8[cur][q]);
          if (live && row_live && done) {
            __stcs(mom_col + (size_t)m * ld, vn);
            __stcs(new_col + (size_t)m * ld, tn);
          }
          v[m] = tn;
          asum += row_live ? tn : 0.f;
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");   // accumulator reads ordered before the next tile's signals
      xchg[h][c] = asum;
      named_bar_sync(2, CONS);                    // column sums published; also: everyone is done with the accumulators
      if (*(volatile int*)&abort_flag) break;
      if (want_cd || a.x_next) {
        const float mean = (asum + xchg[h ^ 1][c]) * invK;
        if (a.x_next && live && h == 0) __stcs(a.x_next + col, mean);
        if (live && want_cd) {
#pragma unroll
          for (int m = 0; m < H; ++m) {
            const float d = v[m] - mean;
            sacc[m] = fmaf(d, d, sacc[m]);
          }
        }
      }
    }
  }

  // ---- wrap-up: tensor memory back, consensus partial sums (box memory is free now)
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == CONS / 32 + 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TcGossipShape<KP>::kTmemCols) : "memory");
  }
  if (want_cd) {
    double* red = reinterpret_cast<double*>(base);    // [CONS/32][H]
    if (warp < CONS / 32) {
#pragma unroll
      for (int m = 0; m < H; ++m) {
        double d = (double)sacc[m];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_down_sync(0xffffffffu, d, off);
        if (lane == 0) red[warp * H + m] = d;
      }
    }
    __syncthreads();
    if (tid < KR) {
      const int hh = tid / H, mm = tid % H;
      double d = 0.0;
#pragma unroll
      for (int w = 0; w < T / 32; ++w) d += red[(hh * (T / 32) + w) * H + mm];
      a.partials[(size_t)blockIdx.x * KR + tid] = d;
    }
    finalize_in_last_cta(a.partials, KR, a.cd_out, a.done);
  }
}

}  // namespace fgd
#endif
