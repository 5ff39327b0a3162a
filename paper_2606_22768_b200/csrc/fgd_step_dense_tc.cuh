// Fused outer step with a DENSE Mix2 on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// For a dense K x K mixing matrix the step ghat[m][p] = sum_n W[m][n] g[n][p] really is a
// contraction (2K flop per worker-parameter; at K = 64 the CUDA-core version is FMA-bound at
// about a quarter of the HBM roofline).  Here it runs as tcgen05.mma.kind::tf32 with the
// error-compensated three-product split
//     W g  ~=  W_hi g_hi + W_hi g_lo + W_lo g_hi          (hi = tf32-rounded, lo = remainder)
// accumulated in fp32 in tensor memory: relative error about 2^-22 of sum |W||g| (the remainders
// are themselves cut to tf32 and the lo x lo term is dropped) -- four times fp32 rounding, well
// inside the 1e-5 parity bar that a single tf32 product would miss.
//
// Mapping.  The 128 columns of a tile are the M dimension of the MMA, the K workers n are its
// K dimension and the K output rows m its N dimension:
//     D[col][m] += A[col][n] * B[n][m],   A = g^T, B = W^T, both K-major (worker-contiguous).
// D row `col` lives in TMEM lane `col`, so after tcgen05.ld the two threads of column `col` hold
// its ghat values in registers -- the same thread-owns-a-column layout as the other kernels;
// the Nesterov update, the streaming stores and the consensus sums follow with one exchange of
// the column sum.
//
// Pipeline per CTA (one per SM): a producer warp streams [K x 128] boxes of theta_prev,
// theta_local and momentum into a shared-memory ring (2 stages at K = 64 and 48, 4 at K = 32)
// with 2-D TMA loads; the eight consumer warps (two threads per column, half of the workers
// each) compute g = theta_prev - theta_local in registers, split it and write g_hi / g_lo IN
// PLACE over the theta_local / theta_prev boxes of the stage in the K-major core-matrix operand
// layout (a thread's four consecutive workers are one 16-byte row of a core matrix, so its
// stores are 128-bit and conflict-free); one thread issues the 3 x (K/8) MMAs and commits them
// to an mbarrier; every consumer then reads its accumulator row from TMEM.
// Worker counts between the shapes are zero-padded (FULL), Mix1 may be given, a fused mean or a
// fused sparse mix (XM), Mix2 may be restricted to column ranges (SUB), and the 32-worker shape
// runs two consumer groups (NG): see the template parameters below.
// All waits are bounded; tensor memory is always released before the kernel returns.
#ifndef FGD_STEP_DENSE_TC_CUH_
#define FGD_STEP_DENSE_TC_CUH_

#include "fgd_step_tma.cuh"

namespace fgd {

__device__ __forceinline__ void named_bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ float to_tf32(float x) {   // round to nearest tf32 (low 13 mantissa bits zero)
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
// Shared-memory matrix descriptor of the tcgen05 MMA (addresses and offsets in 16-byte units).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout_type) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;                  // descriptor version of this architecture
  d |= (uint64_t)(layout_type & 7) << 61;  // 0 = no swizzle, 2 = 128-byte swizzle
  return d;
}
__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
constexpr int kTcMaxK = 64;         // most workers (MMA K and N dimensions)
constexpr int kTcMinK = 17;         // fewest workers sent to this kernel (padding dominates below)
constexpr int kTcCols = 128;        // columns per tile (MMA M dimension)
constexpr int kTcConsumers = 2 * kTcCols;   // two threads share a column, each owns half of the workers
// Shapes.  KP = padded worker count (a multiple of 16: the MMA's N granularity at M = 128);
// worker counts in between are zero-padded up to the next shape.
template <int KP>
struct TcShape {
  static_assert(KP % 16 == 0 && KP >= 32 && KP <= kTcMaxK, "unsupported padded worker count");
  static constexpr int kHalf = KP / 2;                                 // workers per consumer thread
  static constexpr uint32_t kBox = KP * kTcCols * sizeof(float);       // one tensor of a stage
  static constexpr uint32_t kWBytes = KP * KP * sizeof(float);         // one split of W
  static constexpr uint32_t kSbo = KP * 32;                            // operand layout: bytes between 8-row groups
  static constexpr int kTmemCols = KP <= 32 ? 32 : 64;                 // fp32 accumulator columns: a power of two >= 32
  static constexpr int kStages = KP <= 32 ? 4 : 2;                     // what fits in 227 KB next to W_hi and W_lo
  // dynamic shared memory: alignment slack + stages + W_hi + W_lo
  static constexpr size_t kSmem = 128 + (size_t)kStages * 3 * kBox + 2 * kWBytes;
};
constexpr int tc_padded_k(int K) { return K <= 32 ? 32 : (K <= 48 ? 48 : 64); }

// 32 lanes x 32 bit x 8 columns: thread i of the warp receives 8 consecutive columns of lane
// (base + i).  No wait: tmem_ld_wait() makes the registers valid.
__device__ __forceinline__ void tmem_ld_8(uint32_t taddr, float* r) {
  uint32_t* u = reinterpret_cast<uint32_t*>(r);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// N (a multiple of 8) consecutive accumulator columns of this thread's lane.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, float (&r)[N]) {
  static_assert(N % 8 == 0, "column count must be a multiple of 8");
#pragma unroll
  for (int j = 0; j < N; j += 8) tmem_ld_8(taddr + (uint32_t)j, &r[j]);
  tmem_ld_wait();
}

// 32 lanes x 32 bit x 8 columns, registers -> tensor memory (this thread's lane); tmem_st_wait()
// orders the stores before later tensor-memory reads of the same thread.
__device__ __forceinline__ void tmem_st_8(uint32_t taddr, const float* r) {
  const uint32_t* u = reinterpret_cast<const uint32_t*>(r);
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Sparse Mix1 of the rows [r0, r0 + H) of one column from a staged [K][T] box of theta_prev.
// DJ >= the used slot count: unused slots point at the row itself with weight 0, padded rows have
// all-zero weights, so neither needs a branch; all loads of a row are issued before its FMAs.
template <int DJ, int H, int T>
// The H results go to this thread's tensor-memory scratch columns [tx, tx + H), eight at a time:
// they are needed again only in the epilogue, and with all shared memory given to the stages a
// spilled register goes all the way to L2.
__device__ __forceinline__ void tc_gather_x_rows(const GatherMix& m1, const float* A, int r0, int c, uint32_t tx) {
#pragma unroll
  for (int mb = 0; mb < H; mb += 8) {
    float x8[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int r = r0 + mb + q;
      float t[DJ > 0 ? DJ : 1];
#pragma unroll
      for (int j = 0; j < DJ; ++j) t[j] = A[m1.nbr[r * FGD_MAX_D + j] * T + c];
      float acc = m1.w_self[r] * A[r * T + c];
#pragma unroll
      for (int j = 0; j < DJ; ++j) acc = fmaf(m1.w[r * FGD_MAX_D + j], t[j], acc);
      x8[q] = acc;
    }
    tmem_st_8(tx + (uint32_t)mb, x8);
  }
  tmem_st_wait();
}

// The first row of the thread's half as a constant: every neighbour index and weight of the unrolled
// gather is then read at a compile-time offset of the kernel's parameters (an immediate constant-bank
// operand) instead of through an indexed constant load per slot and row.
template <int DJ, int H, int T>
__device__ __forceinline__ void tc_gather_x(const GatherMix& m1, const float* A, int r0, int c, uint32_t tx) {
  if (r0 == 0) tc_gather_x_rows<DJ, H, T>(m1, A, 0, c, tx);
  else tc_gather_x_rows<DJ, H, T>(m1, A, H, c, tx);
}

// XM: where the Mix1 result x comes from.  0 = one value per column (a given row, or the column
// mean of theta_prev computed here); 1 = a given [K, ld] matrix; 2 = a sparse (gossip) Mix1 fused
// into this kernel: x_m = w_self[m] theta_prev[m] + sum_j w[m][j] theta_prev[nbr[m][j]], gathered
// from the theta_prev box of the stage before the operands overwrite it.  (A compile-time switch:
// the per-row x costs up to 32 extra registers per thread, which would slow the common case down.)
// FULL: exactly KP workers.  Otherwise the worker count KR < KP is a run-time value and the
// problem is zero-padded to KP: the TMA boxes stay KP rows tall (rows at or beyond KR are outside
// the tensor and arrive as zeros without touching HBM), W is padded with zero rows and columns,
// and only the first KR rows are stored.
// SUB: Mix2 only on the columns inside the caller's ranges, the identity elsewhere (the thread keeps
// its g values in registers across the MMA and takes them instead of the accumulator row there).
// NG: consumer groups.  With two, group g takes every second tile of the CTA (its own stages,
// named barriers, MMA barrier and accumulator columns), so one group's epilogue -- TMEM read,
// update, stores -- overlaps the other's operand preparation and MMA.  544 threads leave 96
// registers each: that fits the 32-worker shape (measured: K = 17 3.3 -> 4.7 TB/s, K = 24 4.6 ->
// 5.7, dense K = 32 5.4 -> 5.6) and spills at 48 and 64 workers (K = 64: 10.8 -> 13.8 ms), which
// therefore keep one group.
// (registers are handed out per four warps: 288 threads count as 384, i.e. at most 168 registers
// each, and 544 as 640, i.e. 96 -- asking for more makes the kernel unlaunchable)
template <int KP, int XM, bool FULL, bool SUB = false, int NG = 1>
__global__ void __launch_bounds__(NG * kTcConsumers + 32, 1)
outer_step_dense_tc_kernel(const TmaStepArgs ta, const DenseMix m2, const GatherMix m1,
                           const __grid_constant__ CUtensorMap tm_prev, const __grid_constant__ CUtensorMap tm_local,
                           const __grid_constant__ CUtensorMap tm_mom, const __grid_constant__ CUtensorMap tm_x) {
  using Shape = TcShape<KP>;
  constexpr int K = KP, T = kTcCols, H = Shape::kHalf, CONS = kTcConsumers, STAGES = Shape::kStages;
  constexpr uint32_t kTcBox = Shape::kBox, kTcWBytes = Shape::kWBytes, SBO = Shape::kSbo;
  constexpr int ALLC = NG * CONS;                   // all consumer threads; the producer warp follows them
  // tensor memory: the accumulator columns of every group, then as many scratch columns: x of a
  // fused sparse Mix1, or g where Mix2 is restricted to column ranges; 32 + 32, 64 + 64: powers of two
  constexpr int kTmemAll = NG * Shape::kTmemCols * ((XM == 2 || SUB) ? 2 : 1);   // per group: accumulator [+ scratch]
  static_assert(kTmemAll <= 128, "tensor-memory budget of this kernel");
  static_assert(!(XM == 2 && SUB), "one set of scratch columns");
  static_assert(STAGES % NG == 0, "every stage belongs to one group");
  const int KR = FULL ? K : ta.s.K;                 // real worker count (<= K)
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * STAGES + NG];  // full[], empty[], mma[group]
  __shared__ int abort_flag;
  __shared__ uint32_t tmem_base_slot;
  __shared__ float xchg[NG][2][T];   // the two halves of a column exchange their theta_new sums
  // ... and, for a fused global-average Mix1, their theta_prev sums
  __shared__ float xsum[NG][2][T];
  static_assert(NG == 1 || KP < 64, "two groups at 64 workers: no shared memory left for the exchange rows (and no registers)");

  const StepArgs& a = ta.s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gid = (NG > 1 && tid < ALLC) ? tid / CONS : 0;      // consumer group of this thread
  const bool want_cd = a.partials != nullptr;
  unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);   // TMA wants 128-byte alignment
  unsigned char* wb_hi = base + (size_t)STAGES * 3 * kTcBox;
  unsigned char* wb_lo = wb_hi + kTcWBytes;
  const uint32_t mma_bar = smem_u32(&bars[2 * STAGES + gid]);

  const int64_t P = a.P, ld = a.ld;
  const int64_t ntiles = (P + T - 1) / T;

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&bars[s]), 1);
      mbar_init(smem_u32(&bars[STAGES + s]), CONS);
    }
    for (int g = 0; g < NG; ++g) mbar_init(smem_u32(&bars[2 * STAGES + g]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // B operand = W^T as an N x K (m x n) matrix, K-major, no swizzle: 8-row x 16-byte core
  // matrices; core matrices adjacent in K are 128 B apart, adjacent in N SBO = 32 K bytes apart.
  for (int i = tid; i < K * K; i += ALLC + 32) {
    const int n = i / K, m = i % K;          // m2.Wt[n*KR+m] = W[m][n]
    const float w = (FULL || (n < KR && m < KR)) ? m2.Wt[n * KR + m] : 0.f;
    const float hi = to_tf32(w);
    const uint32_t off = (uint32_t)(m >> 3) * SBO + (uint32_t)(n >> 2) * 128u + (uint32_t)(m & 7) * 16u + (uint32_t)(n & 3) * 4u;
    *reinterpret_cast<float*>(wb_hi + off) = hi;
    *reinterpret_cast<float*>(wb_lo + off) = w - hi;
  }
  if (warp == ALLC / 32) {   // the producer warp owns tensor memory: allocate the accumulator columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"((uint32_t)kTmemAll) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // W operands are read by the MMA (async proxy)
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_base_slot;
  const uint32_t tmem_acc = tmem_base + (uint32_t)(gid * Shape::kTmemCols);   // this group's accumulator columns

  float sacc[H];
#pragma unroll
  for (int m = 0; m < H; ++m) sacc[m] = 0.f;

  if (warp == ALLC / 32) {
    // ===================================================== producer (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t i = 0;
      bool ok = true;
      for (int64_t tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++i) {
        const int s = (int)(i % STAGES);
        const uint32_t use = (uint32_t)(i / STAGES);
        if (use > 0) ok = mbar_wait(smem_u32(&bars[STAGES + s]), (use - 1) & 1, ta.spin_limit);
        if (!ok || *(volatile int*)&abort_flag) { ok = false; break; }
        const uint32_t full = smem_u32(&bars[s]);
        mbar_expect_tx(full, 3 * kTcBox);
        if (i == ta.skip_tile) continue;           // test hook: these loads never arrive
        const uint32_t dst = smem_u32(base + (size_t)s * 3 * kTcBox);
        const int c0 = (int)(tile * T);
        tma_load_2d(dst, &tm_prev, c0, 0, full, policy);
        tma_load_2d(dst + kTcBox, &tm_local, c0, 0, full, policy);
        tma_load_2d(dst + 2 * kTcBox, &tm_mom, c0, 0, full, policy);
        // a matrix-valued x is read by the consumers straight into registers: have its box waiting in L2
        if (XM == 1 && ta.n_tensors == 4) tma_prefetch_2d(&tm_x, c0, 0);
      }
      if (!ok) {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      // never exit under a copy in flight: bounded wait for the last use of every stage
      for (int64_t j = (i > STAGES ? i - STAGES : 0); j < i; ++j)
        if (j != ta.skip_tile) mbar_wait(smem_u32(&bars[j % STAGES]), (uint32_t)(j / STAGES) & 1, ta.spin_limit);
    }
  } else {
    // ===================================================== consumers
    // Two threads per column: thread (c, h) owns column c of the tile and the workers
    // [H h, H h + H), H = K / 2 -- eight consumer warps instead of four hide the shared-memory,
    // TMEM and barrier latencies, and half-length arrays keep everything in registers.
    const int lt = tid & (CONS - 1);              // index within the group
    const int c = lt & (T - 1), h = lt >> 7, r0 = h * H;
    const uint32_t tmem_lane = (uint32_t)((warp & 3) * 32) << 16;      // this warp's quarter of the lanes
    // scratch columns of this thread (behind all accumulator columns)
    const uint32_t tmem_x = tmem_base + (uint32_t)((NG + gid) * Shape::kTmemCols) + tmem_lane + (uint32_t)r0;
    const float invK = 1.0f / (float)KR;
    const int hr = FULL ? H : min(max(KR - r0, 0), H);   // live workers of this thread
    const float lr = a.lr, mu = a.mu;
    const bool need_tsum = XM == 0 && a.xsrc == XSRC_FUSED;           // fused mean Mix1
    // A operand = g^T as an M x K (column x worker) matrix, K-major, no swizzle, same core-matrix
    // scheme as B: row c, four consecutive workers = one 16-byte core-matrix row, so a thread's
    // H values go out as H / 4 conflict-free 128-bit stores.
    const uint32_t op_row = (uint32_t)(c >> 3) * SBO + (uint32_t)(c & 7) * 16u;
    // instruction descriptor: D fp32, A and B tf32, both K-major, N = K, M = 128
    constexpr uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(K >> 3) << 17) | ((uint32_t)(T >> 4) << 24);
    int64_t i = gid;                               // the CTA's i-th tile; group g takes i = g, g + NG, ...
    // A one-value-per-column x is requested a whole tile ahead: under a saturated memory system a plain
    // load waits in the same queues as the TMA boxes for several microseconds, longer than the part of a
    // tile that precedes its first use.
    const int64_t tile_step = (int64_t)NG * gridDim.x;
    float x_ahead = 0.f;
    {
      const int64_t col0 = (blockIdx.x + (int64_t)gid * gridDim.x) * T + c;
      if (a.xsrc == XSRC_VECTOR && col0 < P) x_ahead = __ldcs(a.x + col0);
    }
    for (int64_t tile = blockIdx.x + (int64_t)gid * gridDim.x; tile < ntiles; tile += tile_step, i += NG) {
      const int s = (int)(i % STAGES);
      const uint32_t use = (uint32_t)(i / STAGES);
      const int64_t col = tile * T + c;
      const bool live = col < P;
      float xv = x_ahead;
      if (a.xsrc == XSRC_VECTOR && col + tile_step * T < P) x_ahead = __ldcs(a.x + col + tile_step * T);
      float xr[XM == 1 ? H : 1];                   // a matrix-valued Mix1 result: this thread's rows, requested
      if constexpr (XM == 1) {                     // now so that they arrive behind the TMA wait and the MMA
        if (live) {
#pragma unroll
          for (int m = 0; m < H; ++m) xr[m] = (FULL || m < hr) ? __ldcs(a.x + (size_t)(r0 + m) * ld + col) : 0.f;
        }
      }
      unsigned char* stage = base + (size_t)s * 3 * kTcBox;
      float* A = reinterpret_cast<float*>(stage);                 // theta_prev  -> g_lo operand
      float* B = reinterpret_cast<float*>(stage + kTcBox);        // theta_local -> g_hi operand
      float* C = reinterpret_cast<float*>(stage + 2 * kTcBox);    // momentum
      // ---- phase 1: g of this thread's workers in registers
      float g[H];
      float tsum = 0.f;
      const bool got = mbar_wait(smem_u32(&bars[s]), use & 1, ta.spin_limit);
      if (got) {
#pragma unroll
        for (int n = 0; n < H; ++n) {
          const float tp = A[(r0 + n) * T + c];
          g[n] = tp - B[(r0 + n) * T + c];
          tsum += tp;
        }
        if (need_tsum) xsum[gid][h][c] = tsum;          // the column mean needs the other half's sum too
        if constexpr (SUB) {                       // outside the ranges ghat = g: park g next to the accumulator
#pragma unroll
          for (int n = 0; n < H; n += 8) tmem_st_8(tmem_x + (uint32_t)n, &g[n]);
          tmem_st_wait();
        }
        if constexpr (XM == 2) {                   // gossip Mix1 of this thread's rows, from the stage
          const int D1 = m1.D;                     // (uniform) -> a fully unrolled gather per slot count
          if (D1 == 0) tc_gather_x<0, H, T>(m1, A, r0, c, tmem_x);
          else if (D1 == 1) tc_gather_x<1, H, T>(m1, A, r0, c, tmem_x);
          else if (D1 == 2) tc_gather_x<2, H, T>(m1, A, r0, c, tmem_x);
          else if (D1 <= 4) tc_gather_x<4, H, T>(m1, A, r0, c, tmem_x);
          else tc_gather_x<FGD_MAX_D, H, T>(m1, A, r0, c, tmem_x);
        }
      } else {
        *(volatile int*)&abort_flag = 1;
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      named_bar_sync(1 + 3 * gid, CONS);          // every consumer of the group has read its theta_prev / theta_local
      if (*(volatile int*)&abort_flag) break;     // uniform: the flag was written before the barrier
      if (need_tsum) tsum += xsum[gid][h ^ 1][c];
      // ---- operands: g_hi over the theta_local box, g_lo over the theta_prev box
#pragma unroll
      for (int n = 0; n < H; n += 4) {
        float4 hi, lo;
        hi.x = to_tf32(g[n]);     lo.x = g[n] - hi.x;
        hi.y = to_tf32(g[n + 1]); lo.y = g[n + 1] - hi.y;
        hi.z = to_tf32(g[n + 2]); lo.z = g[n + 2] - hi.z;
        hi.w = to_tf32(g[n + 3]); lo.w = g[n + 3] - hi.w;
        const uint32_t off = op_row + (uint32_t)((r0 + n) >> 2) * 128u;
        *reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(B) + off) = hi;
        *reinterpret_cast<float4*>(reinterpret_cast<unsigned char*>(A) + off) = lo;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      named_bar_sync(2 + 3 * gid, CONS);          // operands complete; last tile's TMEM reads are done too
      if (lt == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_hi = smem_u32(B), a_lo = smem_u32(A);
        const uint32_t b_hi = smem_u32(wb_hi), b_lo = smem_u32(wb_lo);
#pragma unroll
        for (int prod = 0; prod < 3; ++prod) {     // W_hi g_hi, W_hi g_lo, W_lo g_hi
          const uint32_t aa = prod == 1 ? a_lo : a_hi;
          const uint32_t bb = prod == 2 ? b_lo : b_hi;
#pragma unroll
          for (int ks = 0; ks < K / 8; ++ks) {
            const uint64_t da = umma_desc(aa + (uint32_t)ks * 256u, 128u, SBO, 0u);
            const uint64_t db = umma_desc(bb + (uint32_t)ks * 256u, 128u, SBO, 0u);
            umma_tf32(tmem_acc, da, db, idesc, (prod | ks) ? 1u : 0u);
          }
        }
        umma_commit(mma_bar);
      }
      // ---- while the tensor core works: this thread's momentum values from the stage
      float v[H];
#pragma unroll
      for (int m = 0; m < H; ++m) v[m] = C[(r0 + m) * T + c];
      if (a.avg_momentum) {                        // GlobalM1S option: v_m <- mean_n v_n (all workers)
        float vs = 0.f;
#pragma unroll
        for (int m = 0; m < H; ++m) vs += v[m] + C[((H - r0) + m) * T + c];
        vs *= invK;
#pragma unroll
        for (int m = 0; m < H; ++m) v[m] = vs;
      }
      if (need_tsum) xv = tsum * invK;
      if (!mbar_wait(mma_bar, (uint32_t)(i / NG) & 1, ta.spin_limit)) {
        *(volatile int*)&abort_flag = 1;          // seen by everyone at the next tile's barrier
        atomicExch(ta.status, FGD_ERR_TIMEOUT);
      }
      // the MMA has consumed the operands and this thread's momentum is in registers: the stage can
      // be refilled while the epilogue below runs from registers and tensor memory
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&bars[STAGES + s]));
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float asum = 0.f;
      if constexpr (XM != 0) {
        // ---- phase 2, per-row x: the accumulator (and the x of a fused sparse Mix1) comes back from
        // tensor memory eight rows at a time, which keeps the full-length register arrays to v /
        // theta_new, the consensus sums and -- for a matrix-valued x -- the prefetched x itself
        float* const mom_col = a.momentum + (size_t)r0 * ld + col;
        float* const new_col = a.theta_new + (size_t)r0 * ld + col;
        float gh8[2][8], x8[2][8];                 // double-buffered: the next eight rows load while these compute
        tmem_ld_8(tmem_acc + tmem_lane + (uint32_t)r0, gh8[0]);
        if constexpr (XM == 2) tmem_ld_8(tmem_x, x8[0]);
#pragma unroll
        for (int mb = 0; mb < H; mb += 8) {
          constexpr int kNext = 8;
          const int cur = (mb / 8) & 1;
          tmem_ld_wait();
          if (mb + kNext < H) {
            tmem_ld_8(tmem_acc + tmem_lane + (uint32_t)(r0 + mb + kNext), gh8[cur ^ 1]);
            if constexpr (XM == 2) tmem_ld_8(tmem_x + (uint32_t)(mb + kNext), x8[cur ^ 1]);
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int m = mb + q;
            const bool row_live = FULL || m < hr;
            const float vn = fmaf(mu, v[m], gh8[cur][q]);
            float xq;
            if constexpr (XM == 2) xq = x8[cur][q];
            else xq = xr[m];
            const float tn = fmaf(-lr, fmaf(mu, vn, gh8[cur][q]), xq);
            if (live && row_live) {
              __stcs(mom_col + (size_t)m * ld, vn);
              __stcs(new_col + (size_t)m * ld, tn);
            }
            v[m] = tn;
            asum += row_live ? tn : 0.f;
          }
        }
      } else {
        float gh[H];                                 // TMEM lane = column, TMEM columns r0.. = this thread's workers
        if constexpr (SUB) {
          // identity on a column outside the ranges: read g back instead of W g.  A tensor-memory
          // load takes ONE address per warp, so the choice is made per warp; the rare warp that
          // straddles a range boundary reads both and selects per thread.
          const bool applies = mix2_applies(a, col);
          const bool any_in = __any_sync(0xffffffffu, applies), all_in = __all_sync(0xffffffffu, applies);
          tmem_ld_cols<H>(any_in ? tmem_acc + tmem_lane + (uint32_t)r0 : tmem_x, gh);
          if (any_in && !all_in) {
#pragma unroll
            for (int n = 0; n < H; n += 8) {
              float t8[8];
              tmem_ld_8(tmem_x + (uint32_t)n, t8);
              tmem_ld_wait();
#pragma unroll
              for (int q = 0; q < 8; ++q) gh[n + q] = applies ? gh[n + q] : t8[q];
            }
          }
        } else {
          tmem_ld_cols<H>(tmem_acc + tmem_lane + (uint32_t)r0, gh);
        }
        // ---- phase 2: Nesterov step for this thread's workers of the column, stream out
        if (live) {
          float* const mom_col = a.momentum + (size_t)r0 * ld + col;
          float* const new_col = a.theta_new + (size_t)r0 * ld + col;
#pragma unroll
          for (int m = 0; m < H; ++m) {
            if (!FULL && m >= hr) break;           // (the per-row-x branch above predicates instead: an
            const float vn = fmaf(mu, v[m], gh[m]);  //  early exit cost those register-heavy variants half their speed)
            const float tn = fmaf(-lr, fmaf(mu, vn, gh[m]), xv);
            __stcs(mom_col + (size_t)m * ld, vn);
            __stcs(new_col + (size_t)m * ld, tn);
            v[m] = tn;
            asum += tn;
          }
        }
      }
      if (want_cd || a.x_next) {                   // column mean over both halves, then squared deviations
        xchg[gid][h][c] = asum;
        named_bar_sync(3 + 3 * gid, CONS);
        const float mean = (asum + xchg[gid][h ^ 1][c]) * invK;
        if (a.x_next && live && h == 0) __stcs(a.x_next + col, mean);   // next round's global-average Mix1
        if (live && want_cd) {
#pragma unroll
          for (int m = 0; m < H; ++m) {            // (sums of padded rows are never read)
            const float d = v[m] - mean;
            sacc[m] = fmaf(d, d, sacc[m]);
          }
        }
      }
    }
  }

  // ---- wrap-up: tensor memory back, consensus partial sums (stage memory is free now)
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == ALLC / 32) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemAll) : "memory");
  }
  if (want_cd) {
    double* red = reinterpret_cast<double*>(base);    // [ALLC/32][H]; per group: warps 0-3 hold the first half of the workers, 4-7 the second
    if (warp < ALLC / 32) {
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
      for (int g = 0; g < NG; ++g)
#pragma unroll
        for (int w = 0; w < T / 32; ++w) d += red[((g * 2 + hh) * (T / 32) + w) * H + mm];
      a.partials[(size_t)blockIdx.x * KR + tid] = d;
    }
    finalize_in_last_cta(a.partials, KR, a.cd_out, a.done);
  }
}

}  // namespace fgd
#endif
