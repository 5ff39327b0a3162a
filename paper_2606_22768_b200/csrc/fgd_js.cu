// JS functional-disagreement metric CD_JS (the paper's App. D.2) on logits resident in HBM.
//
// Per token position u: the top_k tokens of the parameter-averaged model's logits are selected
// (exact radix select, ties to the lower token index); every worker's distribution and the
// averaged model's are restricted to those tokens, renormalised, and compared with the
// normalised Jensen-Shannon distance sqrt(JS / ln 2), all in float64 in the log domain.
// Kernels: one CTA per position selects the tokens in a single pass over the row (rows that defeat
// its sampling bound are redone by an exact multi-pass select), one warp per (worker, position)
// pair evaluates the distance, and a last kernel sums the distances of each worker in a fixed order.
#include <cuda_runtime.h>

#include <cstdio>

#include "fgd_internal.h"
#include "fgd_nvtx.h"
#include "fgd_step_dense_tc.cuh"   // mbarrier / shared-memory helpers

using namespace fgd;

namespace {

constexpr int kSelBlock = 1024;
constexpr int kMaxTopK = 256;

int js_fail(int status, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_thread_error, sizeof(g_thread_error), fmt, ap);
  va_end(ap);
  return status;
}

// fp32 -> unsigned key whose ASCENDING order is DESCENDING float order (largest logit first).
// (ascending key = negative ? ~b : b | sign; its complement in two operations)
__device__ __forceinline__ uint32_t desc_key(float x) {
  const uint32_t b = __float_as_uint(x);
  const uint32_t neg = (uint32_t)((int32_t)b >> 31);      // all ones for a negative value
  return b ^ (~neg & 0x7FFFFFFFu);
}

// ---------------------------------------------------------------------------------------------
// Streaming select: ONE pass over the row in HBM.
//
// A lower bound of the k-th largest logit of the whole row comes from a sample: every thread takes
// the largest of its 24 elements of the row's first 12 K, and the k-th largest of those 512 maxima
// bounds the row's k-th largest from below (k distinct elements reach it).  It is located on a 12-bit
// histogram of the ordered keys (sign, exponent, three mantissa bits) and then sharpened to the exact
// key by ranking the few maxima of the boundary bin.  The row is then streamed once; four elements at a
// time are compared with the bound as floats, and the rare elements that reach it (about one percent
// of a row in random order) are appended to a candidate list in shared memory.  The exact answer --
// the k smallest (key, index) pairs, i.e. ties to the lower token index -- is found among the
// candidates: a second histogram over them gives the row's true boundary bin, whatever lies before
// it is selected, and each member of the boundary bin counts how many members precede it as a
// (key, index) pair to learn whether it is among the few still needed; the k indices find their
// output slots the same way (rank by counting: no sorting network).
// A row that defeats the sample (ascending order, huge groups of equal logits) overflows a list; it
// is then marked (first output index -1) and redone by the exact multi-pass kernel below.
// The row travels through two 24 KB shared-memory stages filled by 1-D bulk copies (TMA) that a
// producer warp keeps in flight, so the bytes in flight do not depend on the consumers' registers;
// the first two stages double as the sample (they are looked at twice without being loaded twice).
// Measured: the hand-off per stage, not the bytes, is what costs -- six 8 KB stages 0.84 ms, three
// 16 KB 0.68 ms, two 24 KB 0.62 ms, one 48 KB 0.68 ms for the whole call at U = 4096 -- and three CTAs
// per SM (69 KB each) beat two with a larger ring, because one row's start-up and candidate phases
// then overlap two other rows' streaming.
constexpr int kStrConsumers = 512;             // consumer threads; one more warp produces
constexpr int kStrBlock = kStrConsumers + 32;
constexpr int kBinShift = 20;                  // key >> 20: 4096 bins (sign, exponent, three mantissa bits)
constexpr int kBins = 1 << (32 - kBinShift);
constexpr int kChunk = 6144;                   // floats per stage (24 KB)
constexpr int kStrStages = 2;                  // the ring; also the sample (12 K elements)
constexpr int kCand = 2048;                    // candidate list entries
constexpr int kBnd = 512;                      // boundary-bin list entries
// The histogram has no memory of its own: for the sample it lies over the (still empty) candidate
// list, for the candidates over the (by then idle) ring -- 69 KB per CTA, three CTAs per SM, so that one
// row's start-up and candidate phases overlap two other rows' streaming.
static_assert(sizeof(unsigned) * kBins <= sizeof(unsigned long long) * kCand && sizeof(unsigned) * kBins <= sizeof(float) * kChunk * kStrStages,
              "the histogram must fit over the candidate list and over the ring");
constexpr size_t kStrSmem = 128 + sizeof(float) * kChunk * kStrStages +
                            sizeof(unsigned long long) * (kCand + kBnd) + sizeof(int) * kMaxTopK;
constexpr uint32_t kStrSpin = 1u << 22;        // polls before a wait gives up (the row is then redone by the exact kernel)

__device__ __forceinline__ bool js_wait(uint32_t bar, uint32_t parity, const int* abort_flag) {
  for (uint32_t it = 0; it < kStrSpin; ++it) {
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

// One lane polls, the warp follows (far fewer polls competing with the other CTA's arithmetic).
__device__ __forceinline__ bool js_warp_wait(uint32_t bar, uint32_t parity, const int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = js_wait(bar, parity, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// First bin b with cum(b) >= k over hist[kBins]; the kStrConsumers consumer threads call (named
// barrier 1).  *bin_out, *before_out: that bin and the count of the bins before it; untouched when
// the histogram holds fewer than k entries.
__device__ __forceinline__ void find_boundary_bin(const unsigned* hist, unsigned k, unsigned* warp_tot, unsigned* bin_out,
                                                  unsigned* before_out, int tid) {
  constexpr int PER = kBins / kStrConsumers;
  const int lane = tid & 31, warp = tid >> 5;
  unsigned loc[PER], sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { loc[j] = hist[tid * PER + j]; sum += loc[j]; }
  unsigned incl = sum;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned t = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += t;
  }
  if (lane == 31) warp_tot[warp] = incl;
  named_bar_sync(1, kStrConsumers);
  unsigned before = incl - sum;
  for (int w = 0; w < warp; ++w) before += warp_tot[w];
  if (before < k && before + sum >= k) {       // exactly one thread, unless the total is below k
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (before < k && before + loc[j] >= k) { *bin_out = (unsigned)(tid * PER + j); *before_out = before; }
      before += loc[j];
    }
  }
  named_bar_sync(1, kStrConsumers);
}

__global__ void __launch_bounds__(kStrBlock)
js_select_stream_kernel(const float* __restrict__ avg_logits, int64_t V, int k, int32_t* __restrict__ idx_out) {
  extern __shared__ __align__(128) unsigned char js_smem[];
  __shared__ __align__(8) unsigned long long bars[2 * kStrStages];     // full[], empty[]
  __shared__ unsigned warp_tot[kStrConsumers / 32];
  __shared__ unsigned s_bin, s_before, s_ncand, s_nbnd, s_nfin, s_keymax;
  __shared__ int abort_flag;
  unsigned char* base = js_smem + ((128u - (smem_u32(js_smem) & 127u)) & 127u);
  float* ring = reinterpret_cast<float*>(base);
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(ring + (size_t)kChunk * kStrStages);
  unsigned* const hist_sample = reinterpret_cast<unsigned*>(cand);     // before any candidate exists
  unsigned* const hist_cand = reinterpret_cast<unsigned*>(ring);       // after the last chunk has been read
  unsigned long long* bnd = cand + kCand;
  int* fin = reinterpret_cast<int*>(bnd + kBnd);
  const float* row = avg_logits + (size_t)blockIdx.x * V;
  int32_t* out = idx_out + (size_t)blockIdx.x * k;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[kStrStages]);

  // the 16-byte aligned body of the row goes through the ring; up to three elements before and
  // after it are read directly
  int64_t head = (int64_t)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(row) & 15u)) & 15u) >> 2);
  if (head > V) head = V;
  const int64_t body = (V - head) / 4 * 4;                 // floats
  const int64_t nchunks = (body + kChunk - 1) / kChunk;
  const int nres = (int)(nchunks < kStrStages ? nchunks : kStrStages);   // chunks resident at the start = the sample

  if (tid == 0) {
    for (int s = 0; s < kStrStages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, kStrConsumers / 32);   // one arrival per consumer warp
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_bin = kBins - 1; s_before = 0; s_ncand = 0; s_nbnd = 0; s_nfin = 0;
    abort_flag = 0;
  }
  for (int i = tid; i < kBins; i += kStrBlock) hist_sample[i] = 0;
  __syncthreads();

  if (warp == kStrConsumers / 32) {
    // ===================================================== producer (one elected lane)
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      int64_t c = 0;
      bool ok = true;
      for (; c < nchunks; ++c) {
        const int s = (int)(c % kStrStages);
        if (c >= kStrStages) ok = js_wait(bar_empty + 8u * s, (uint32_t)(c / kStrStages - 1) & 1, &abort_flag);
        if (!ok) break;
        const int64_t left = body - c * kChunk;
        const uint32_t bytes = (uint32_t)((left < kChunk ? left : kChunk) * sizeof(float));
        mbar_expect_tx(bar_full + 8u * s, bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                     ::"r"(smem_u32(ring + (size_t)s * kChunk)), "l"(row + head + c * kChunk), "r"(bytes), "r"(bar_full + 8u * s), "l"(policy)
                     : "memory");
      }
      if (!ok) *(volatile int*)&abort_flag = 1;
      // never exit under a copy in flight: bounded wait for the last use of every stage
      for (int64_t j = (c > kStrStages ? c - kStrStages : 0); j < c; ++j) {
        const uint32_t bar = bar_full + 8u * (uint32_t)(j % kStrStages), parity = (uint32_t)(j / kStrStages) & 1;
        for (uint32_t it = 0; it < kStrSpin; ++it) {
          uint32_t done;
          asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
          if (done) break;
        }
      }
    }
    return;
  }

  // ===================================================== consumers
  bool failed = false;
  // ---- sample: the largest element each thread sees in the resident chunks
  uint32_t best = 0xFFFFFFFFu;                       // smallest key = largest logit
  bool have = false;
  for (int c = 0; c < nres && !failed; ++c) {
    if (!js_warp_wait(bar_full + 8u * c, 0, &abort_flag, lane)) { failed = true; break; }
    const int64_t left = body - (int64_t)c * kChunk;
    const int n4 = (int)((left < kChunk ? left : kChunk) / 4);
    const float4* src = reinterpret_cast<const float4*>(ring + (size_t)c * kChunk);
    for (int j = tid; j < n4; j += kStrConsumers) {
      const float4 t = src[j];
      best = min(min(best, desc_key(t.x)), min(desc_key(t.y), min(desc_key(t.z), desc_key(t.w))));
      have = true;
    }
  }
  if (have) atomicAdd(&hist_sample[best >> kBinShift], 1u);
  if (failed) *(volatile int*)&abort_flag = 1;
  named_bar_sync(1, kStrConsumers);
  find_boundary_bin(hist_sample, (unsigned)k, warp_tot, &s_bin, &s_before, tid);
  const unsigned b0 = s_bin;
  // The bound is sharpened from "bin b0" to the exact key inside it: the maxima that fall into b0 (a
  // handful) are listed and the (k - before)-th smallest of them, found by counting ranks, is the
  // k-th largest maximum itself.  (If the list overflows the whole bin stays in.)
  const unsigned need0 = (unsigned)k - s_before, nb0 = hist_sample[b0];
  uint32_t* const lst = reinterpret_cast<uint32_t*>(bnd);
  if (tid == 0) s_keymax = b0 >= (unsigned)(kBins - 1) ? 0xFFFFFFFFu : (((b0 + 1u) << kBinShift) - 1u);   // largest key inside bin b0
  named_bar_sync(1, kStrConsumers);
  const bool refine = b0 < (unsigned)(kBins - 1) && nb0 >= need0 && nb0 <= (unsigned)(2 * kBnd);
  const bool mine_in = refine && have && (best >> kBinShift) == b0;
  if (mine_in) lst[atomicAdd(&s_nbnd, 1u)] = best;
  named_bar_sync(1, kStrConsumers);
  if (mine_in) {
    unsigned smaller = 0, equal = 0;
    for (unsigned j = 0; j < nb0; ++j) {
      const uint32_t o = lst[j];
      smaller += o < best ? 1u : 0u;
      equal += o == best ? 1u : 0u;
    }
    if (smaller < need0 && smaller + equal >= need0) s_keymax = best;     // every thread that hits it writes the same key
  }
  named_bar_sync(1, kStrConsumers);
  const uint32_t key_max = s_keymax;
  if (tid == 0) s_nbnd = 0;

  // The same bound as a float: the smallest value of bin b0.  Four elements at a time are tested against
  // it with one comparison of their maximum; only the rare group that reaches it is looked at element
  // by element with the exact key test.  (NaN logits are not supported: fmaxf drops them.)
  float thr;
  {
    const uint32_t bits = (key_max & 0x80000000u) ? key_max : (key_max ^ 0x7FFFFFFFu);   // inverse of desc_key
    thr = __uint_as_float(bits);
    if (key_max == 0xFFFFFFFFu || thr != thr) thr = key_max == 0xFFFFFFFFu ? -__int_as_float(0x7f800000) : __int_as_float(0x7f800000);
  }
  // ---- the one pass over the row: keep what is not beyond the sample's boundary bin
  auto consider = [&](float x, int64_t i) {
    const uint32_t key = desc_key(x);
    if (key <= key_max) {
      const unsigned slot = atomicAdd(&s_ncand, 1u);
      if (slot < (unsigned)kCand) cand[slot] = ((unsigned long long)key << 32) | (unsigned long long)(uint32_t)i;
    }
  };
  if (tid < head) consider(row[tid], tid);
  if (head + body + tid < V) consider(row[head + body + tid], head + body + tid);
  for (int64_t c = 0; c < nchunks && !*(volatile int*)&abort_flag; ++c) {
    const int s = (int)(c % kStrStages);
    if (c >= nres && !js_warp_wait(bar_full + 8u * s, (uint32_t)(c / kStrStages) & 1, &abort_flag, lane)) {
      *(volatile int*)&abort_flag = 1;
      break;
    }
    const int64_t left = body - c * kChunk;
    const int n4 = (int)((left < kChunk ? left : kChunk) / 4);
    const float4* src = reinterpret_cast<const float4*>(ring + (size_t)s * kChunk);
    const int64_t i0 = head + c * kChunk;
#pragma unroll 2
    for (int j = tid; j < n4; j += kStrConsumers) {
      const float4 t = src[j];
      if (fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w)) >= thr) {
        consider(t.x, i0 + 4 * j);
        consider(t.y, i0 + 4 * j + 1);
        consider(t.z, i0 + 4 * j + 2);
        consider(t.w, i0 + 4 * j + 3);
      }
    }
    __syncwarp();                                   // (reads through the generic proxy are ordered before the
    if (lane == 0) mbar_arrive(bar_empty + 8u * s); //  refill by the arrive / wait pair itself: no proxy fence)
  }
  named_bar_sync(1, kStrConsumers);               // every consumer is through with the ring
  for (int i = tid; i < kBins; i += kStrConsumers) hist_cand[i] = 0;
  named_bar_sync(1, kStrConsumers);
  const unsigned ncand = s_ncand;
  if (*(volatile int*)&abort_flag || ncand > (unsigned)kCand) {   // a wait gave up, or the sample's bound was too weak for this row
    if (tid == 0) out[0] = -1;
    return;
  }
  // ---- exact boundary bin of the whole row, from the candidates
  for (unsigned i = tid; i < ncand; i += kStrConsumers) atomicAdd(&hist_cand[(unsigned)(cand[i] >> (32 + kBinShift))], 1u);
  named_bar_sync(1, kStrConsumers);
  find_boundary_bin(hist_cand, (unsigned)k, warp_tot, &s_bin, &s_before, tid);
  const unsigned b1 = s_bin, above = s_before, nb = hist_cand[b1];
  if (nb > (unsigned)kBnd) {                     // too many logits in one bin (large groups of equal values)
    if (tid == 0) out[0] = -1;
    return;
  }
  for (unsigned i = tid; i < ncand; i += kStrConsumers) {
    const unsigned long long e = cand[i];
    const unsigned bin = (unsigned)(e >> (32 + kBinShift));
    if (bin < b1) fin[atomicAdd(&s_nfin, 1u)] = (int)(uint32_t)e;            // selected for certain (above < k of them)
    else if (bin == b1) bnd[atomicAdd(&s_nbnd, 1u)] = e;
  }
  named_bar_sync(1, kStrConsumers);
  // of the boundary bin's nb members the `need` smallest (key, index) pairs are taken: larger logit
  // first, then the lower index.  All pairs are distinct, so a member's rank is the count of smaller ones.
  const unsigned need = (unsigned)k - above;     // 1 <= need <= nb
  for (unsigned i = tid; i < nb; i += kStrConsumers) {
    const unsigned long long e = bnd[i];
    unsigned rank = 0;
    for (unsigned j = 0; j < nb; ++j) rank += bnd[j] < e ? 1u : 0u;
    if (rank < need) fin[above + rank] = (int)(uint32_t)e;
  }
  named_bar_sync(1, kStrConsumers);
  // ---- output in ascending index order: the slot of an index is the count of smaller selected indices
  if (tid < k) {
    const int mine = fin[tid];
    int rank = 0;
    for (int j = 0; j < k; ++j) rank += fin[j] < mine ? 1 : 0;
    out[rank] = mine;
  }
}

// Exact multi-pass select (four 8-bit radix passes and an ordered compaction), one CTA per row.
// Rows the streaming kernel could not finish are marked with a first index of -1; with
// `only_marked` every other row is skipped.
__device__ __forceinline__ void js_select_row(const float* __restrict__ row, int64_t V, int k, int32_t* __restrict__ out) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining, s_less;
  __shared__ unsigned int warp_tot[2][kSelBlock / 32];
  __shared__ unsigned int s_eq_base, s_sel_base;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    s_prefix = 0;
    s_remaining = (unsigned)k;
    s_less = 0;
  }
  // ---- radix select, 8 bits per pass from the top: key of the k-th smallest
  for (int pass = 3; pass >= 0; --pass) {
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    const unsigned prefix = s_prefix;
    const unsigned hi_mask = pass == 3 ? 0u : (0xFFFFFFFFu << (8 * (pass + 1)));
#pragma unroll 4
    for (int64_t i = tid; i < V; i += kSelBlock) {
      const uint32_t key = desc_key(row[i]);
      if ((key & hi_mask) == (prefix & hi_mask)) atomicAdd(&hist[(key >> (8 * pass)) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned cum = 0, rem = s_remaining;
      int b = 0;
      for (; b < 256; ++b) {
        if (cum + hist[b] >= rem) break;
        cum += hist[b];
      }
      s_prefix = prefix | ((unsigned)b << (8 * pass));
      s_remaining = rem - cum;     // rank of the target inside bucket b
      s_less += cum;               // keys known to be smaller than the target
    }
    __syncthreads();
  }
  const unsigned target = s_prefix;
  const unsigned need_eq = (unsigned)k - s_less;   // how many keys equal to the target are taken
  if (tid == 0) {
    s_eq_base = 0;
    s_sel_base = 0;
  }
  __syncthreads();
  // ---- ordered compaction: selected = key < target, or key == target among the first need_eq
  for (int64_t base = 0; base < V; base += kSelBlock) {
    const int64_t i = base + tid;
    uint32_t key = 0xFFFFFFFFu;
    bool valid = i < V;
    if (valid) key = desc_key(row[i]);
    const bool is_eq = valid && key == target;
    // almost every chunk of a large vocabulary holds no candidate at all: one barrier and move on
    if (!__syncthreads_or(valid && key <= target)) continue;
    // block-wide exclusive scan of is_eq
    const unsigned eq_ballot = __ballot_sync(0xffffffffu, is_eq);
    if (lane == 0) warp_tot[0][warp] = __popc(eq_ballot);
    __syncthreads();
    unsigned eq_before = __popc(eq_ballot & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) eq_before += warp_tot[0][w];
    const unsigned eq_rank = s_eq_base + eq_before;
    const bool sel = valid && (key < target || (is_eq && eq_rank < need_eq));
    const unsigned sel_ballot = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) warp_tot[1][warp] = __popc(sel_ballot);
    __syncthreads();
    unsigned sel_before = __popc(sel_ballot & ((1u << lane) - 1u));
    unsigned eq_total = 0, sel_total = 0;
    for (int w = 0; w < kSelBlock / 32; ++w) {
      if (w < warp) sel_before += warp_tot[1][w];
      eq_total += warp_tot[0][w];
      sel_total += warp_tot[1][w];
    }
    if (sel) out[s_sel_base + sel_before] = (int32_t)i;
    __syncthreads();
    if (tid == 0) {
      s_eq_base += eq_total;
      s_sel_base += sel_total;
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kSelBlock)
js_select_kernel(const float* __restrict__ avg_logits, int64_t U, int64_t V, int k, int32_t* __restrict__ idx_out, int only_marked) {
  // a small grid walks the rows: with `only_marked` almost every row costs one load of its marker
  for (int64_t u = blockIdx.x; u < U; u += gridDim.x) {
    if (only_marked && idx_out[(size_t)u * k] != -1) continue;          // (uniform for the CTA)
    js_select_row(avg_logits + (size_t)u * V, V, k, idx_out + (size_t)u * k);
    __syncthreads();                                                    // the shared state is free for the next row
  }
}

__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, off));
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {   // fixed butterfly: every lane gets the same bits
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// One warp per (worker m, position u): normalised JS distance over the selected tokens.
// PER = tokens per lane (k <= 32 PER): the register arrays are sized for the k in use.
template <int PER>
__global__ void __launch_bounds__(256)
js_distance_kernel(const float* __restrict__ worker_logits, const float* __restrict__ avg_logits,
                   const int32_t* __restrict__ idx, int K, int64_t U, int64_t V, int k, double* __restrict__ d_js) {
  const int64_t pair = (int64_t)blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (pair >= (int64_t)K * U) return;
  const int lane = threadIdx.x & 31;
  const int64_t m = pair / U, u = pair - m * U;
  const float* wrow = worker_logits + ((size_t)m * U + u) * V;
  const float* arow = avg_logits + (size_t)u * V;
  const int32_t* id = idx + (size_t)u * k;
  double p[PER], q[PER];
  double pmax = -1e300, qmax = -1e300;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int t = lane + 32 * j;
    if (t < k) {
      const int32_t tok = id[t];
      p[j] = (double)wrow[tok];
      q[j] = (double)arow[tok];
      pmax = fmax(pmax, p[j]);
      qmax = fmax(qmax, q[j]);
    }
  }
  pmax = warp_max(pmax);
  qmax = warp_max(qmax);
  double ps = 0.0, qs = 0.0;
  double ep[PER], eq[PER];                 // exp(logit - max): the probabilities up to their normalising sums
#pragma unroll
  for (int j = 0; j < PER; ++j)
    if (lane + 32 * j < k) {
      ep[j] = exp(p[j] - pmax);
      eq[j] = exp(q[j] - qmax);
      ps += ep[j];
      qs += eq[j];
    }
  ps = warp_sum(ps);
  qs = warp_sum(qs);
  const double plse = pmax + log(ps), qlse = qmax + log(qs);
  const double half_ip = 0.5 / ps, half_iq = 0.5 / qs;
  const double ln_half = -0.69314718055994530942;
  double js = 0.0;
#pragma unroll
  for (int j = 0; j < PER; ++j)
    if (lane + 32 * j < k) {
      const double lp = p[j] - plse, lq = q[j] - qlse;
      const double hi = fmax(lp, lq), lo = fmin(lp, lq);
      const double lm = hi + log1p(exp(lo - hi)) + ln_half;      // log((p + q) / 2)
      js += ep[j] * half_ip * (lp - lm) + eq[j] * half_iq * (lq - lm);   // 1/2 p (log p - log m) + 1/2 q (log q - log m)
    }
  js = warp_sum(js);
  if (lane == 0) d_js[pair] = sqrt(fmax(js, 0.0) / 0.69314718055994530942);
}

// cd_worker[m] = (1/U) sum_u d_js[m][u], one warp per worker, fixed order.
__global__ void __launch_bounds__(32)
js_mean_kernel(const double* __restrict__ d_js, int64_t U, double* __restrict__ cd_worker) {
  const int m = blockIdx.x, lane = threadIdx.x;
  double s = 0.0;
  for (int64_t u = lane; u < U; u += 32) s += d_js[(size_t)m * U + u];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xffffffffu, s, off);
  if (lane == 0) cd_worker[m] = s / (double)U;
}

}  // namespace

extern "C" int fgd_js_distance(int device, int K, int64_t U, int64_t V, int top_k, const float* worker_logits,
                               const float* avg_logits, int32_t* top_idx, double* d_js, double* cd_worker,
                               void* stream) {
  FGD_NVTX_RANGE("fgd_js_distance");
  if (K < 1 || K > FGD_MAX_K || U < 1 || V < 1 || top_k < 1 || top_k > kMaxTopK || top_k > V)
    return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: need 1 <= K <= %d, U, V >= 1, 1 <= top_k <= min(%d, V)", FGD_MAX_K, kMaxTopK);
  if (U * (int64_t)K > 0x7fffffff * 8ll || U > 0x7fffffff || V > 0x7fffffff)
    return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: too many positions");
  if (!worker_logits || !avg_logits || !top_idx || !d_js || !cd_worker) return js_fail(FGD_ERR_INVALID_ARG, "fgd_js_distance: NULL pointer");
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return js_fail(FGD_ERR_CUDA, "cudaGetDevice failed");
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return js_fail(FGD_ERR_CUDA, "cannot select device %d", device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  static bool smem_set[64] = {};
  if (device < 64 && !smem_set[device]) {
    if (cudaFuncSetAttribute(js_select_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStrSmem) != cudaSuccess) {
      if (prev != device) cudaSetDevice(prev);
      return js_fail(FGD_ERR_CUDA, "fgd_js_distance: cannot size the select kernel's shared memory");
    }
    smem_set[device] = true;
  }
  js_select_stream_kernel<<<(unsigned)U, kStrBlock, kStrSmem, st>>>(avg_logits, V, top_k, top_idx);
  js_select_kernel<<<(unsigned)(U < 296 ? U : 296), kSelBlock, 0, st>>>(avg_logits, U, V, top_k, top_idx, 1);   // rows the stream kernel marked
  const int64_t pairs = (int64_t)K * U;
  const unsigned grid_d = (unsigned)((pairs + 7) / 8);
  if (top_k <= 32) js_distance_kernel<1><<<grid_d, 256, 0, st>>>(worker_logits, avg_logits, top_idx, K, U, V, top_k, d_js);
  else if (top_k <= 64) js_distance_kernel<2><<<grid_d, 256, 0, st>>>(worker_logits, avg_logits, top_idx, K, U, V, top_k, d_js);
  else if (top_k <= 128) js_distance_kernel<4><<<grid_d, 256, 0, st>>>(worker_logits, avg_logits, top_idx, K, U, V, top_k, d_js);
  else js_distance_kernel<kMaxTopK / 32><<<grid_d, 256, 0, st>>>(worker_logits, avg_logits, top_idx, K, U, V, top_k, d_js);
  js_mean_kernel<<<K, 32, 0, st>>>(d_js, U, cd_worker);
  cudaError_t e = cudaGetLastError();
  if (prev != device) cudaSetDevice(prev);
  if (e != cudaSuccess) return js_fail(FGD_ERR_CUDA, "fgd_js_distance: launch failed: %s", cudaGetErrorString(e));
  return FGD_OK;
}
