/*
 * fgd.h -- C ABI of the B200 (sm_100a) implementation of the Factored Gossip DiLoCo
 * outer synchronisation round, computed for all K simulated workers on one GPU.
 *
 * Data model.  Worker m's flat parameters are row m of a row-major fp32 matrix
 * [K, ld] (ld >= P, in elements) in DEVICE memory: theta_prev = z_{m,r} (result of the
 * previous outer step, start of the inner loop), theta_local = y_{m,r,H} (after the H
 * inner steps), momentum = v_{m,r} (Nesterov outer momentum), theta_new = z_{m,r+1}.
 * The paper stacks workers as columns X in R^{d x M}; this is the transpose, so
 * "communication" between workers is a read of another row of the same matrix.
 *
 * One round (Sec. 4.1 round equations; Algorithm 1):
 *     x_m      = Mix1(theta_prev)_m                    non-blocking mix, side stream
 *     g_m      = theta_prev_m - theta_local_m          = -Delta_m (outer gradient)
 *     ghat_m   = Mix2(g)_m                             blocking mix
 *     v'_m     = mu v_m + ghat_m                       Nesterov SGD, App. B
 *     theta_new_m = x_m - gamma (ghat_m + mu v'_m)
 *     s_m      = sum_p (theta_new[m][p] - mean_p)^2    consensus distance, Sec. 4.4 / App. D
 * Mix_W(v)_m = sum_n W[m][n] v_n with W symmetric and doubly stochastic (Sec. 3): ROW
 * convention, row m of W = the weights worker m applies.
 *
 * Conventions for every function.
 *  - Every entry point that launches work is wrapped in an NVTX range carrying its own name.
 *  - Returns FGD_OK (0) or a negative fgd_status.  Never throws, aborts, exits or prints.
 *    fgd_last_error() gives a human-readable reason for the last failure on that context.
 *  - Pointers named theta_*, momentum, g, in, out, x, cd_sumsq are DEVICE pointers on the
 *    context's device; everything inside fgd_mix_desc and every argument of the host helpers
 *    (fgd_topo_*, fgd_edge_mask, fgd_effective_weights, fgd_dense_matrix, fgd_cd_finalize) is
 *    HOST memory.
 *  - Ownership: the caller owns all tensors.  The library allocates no parameter-sized
 *    memory and keeps no caller pointer after a call returns; descriptors are consumed
 *    (copied into the launch) before the call returns.
 *  - Calls are asynchronous on `stream` (a cudaStream_t passed as void*, NULL = default
 *    stream): tensors must stay alive until the stream reaches that point.
 *  - Fast path: base pointers 16-byte aligned and ld % 4 == 0; otherwise an element-wise
 *    path is used (slower, not an error).  FULL speed needs rows that start on 128-byte
 *    boundaries (128-byte aligned bases, ld % 32 == 0): every kernel moves 512-byte to 4-KB row
 *    segments, and a segment that starts inside a 32-byte DRAM sector leaves partly written
 *    sectors at both ends.  Measured on the fused step (4 GB per tensor): ld % 32 == 0 -> 1.00;
 *    ld % 8 == 0 only -> 0.97 (8 and 16 workers) to 0.90 (64 workers); ld % 4 == 0 only -> 0.91
 *    (16 workers) to 0.65-0.70 (40 and 64 workers).  The caller owns the layout: pad ld.
 *  - Deterministic: the same inputs give bit-identical outputs (no floating-point atomics).
 *  - Threads: a context is NOT re-entrant.  It carries the last error string, an occupancy cache
 *    and (during fgd_outer_step_from_host) a temporarily narrowed column count, so one context
 *    must be used by one host thread at a time; different contexts are independent.
 *  - fgd_outer_step (with cd_sumsq) and fgd_consensus_distance use the context's small
 *    partial-sum scratch: two such calls on one context must be ordered on the GPU
 *    (same stream or an event); all other calls may overlap freely.
 *  - Stream capture: after one eager call with the same context, mix kind and argument
 *    shapes (it sizes the launch), fgd_outer_grad, fgd_mix, fgd_outer_step(_ex) and
 *    fgd_consensus_distance only enqueue kernels on `stream` -- no allocation, copy or
 *    synchronisation -- so they can be recorded into a CUDA graph.  The descriptors are
 *    kernel arguments: a graph replays the mixes it was captured with.
 */
#ifndef FGD_H_
#define FGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FGD_MAX_K 64 /* most workers (rows) */
#define FGD_MAX_D 8  /* most neighbour slots per worker in a sparse mix */
#define FGD_MAX_RANGES 8 /* most column ranges of a subset Mix2 */
#define FGD_MAX_CHUNKS 32 /* most column chunks of fgd_outer_step_from_host */

typedef enum {
  FGD_OK = 0,
  FGD_ERR_INVALID_ARG = -1, /* NULL pointer, size out of range, malformed descriptor */
  FGD_ERR_ALIGNMENT = -2,   /* reserved: misalignment is handled by the element-wise path */
  FGD_ERR_ALIAS = -3,       /* forbidden overlap between tensors */
  FGD_ERR_UNSUPPORTED = -4, /* valid request this build has no kernel for */
  FGD_ERR_CUDA = -5,        /* a CUDA runtime call failed (message holds the CUDA error) */
  FGD_ERR_TIMEOUT = -6      /* a bounded device-side wait gave up (see fgd_device_status) */
} fgd_status;

typedef struct fgd_ctx fgd_ctx; /* opaque; owns O(#CTAs * K) doubles of device scratch */

/* Create a context for [K, ld] matrices with P used columns on CUDA device `device`.
 * 1 <= K <= FGD_MAX_K, 1 <= P <= ld.  Allocates the partial-sum scratch (about 1 MB). */
int fgd_create(fgd_ctx** out, int device, int K, int64_t P, int64_t ld);
int fgd_destroy(fgd_ctx* ctx);
/* Reason of the last failing call on ctx ("" if none); NULL ctx gives the reason of the
 * last failing fgd_create / host helper on this thread.  The string is owned by the library. */
const char* fgd_last_error(const fgd_ctx* ctx);
const char* fgd_status_string(int status);
/* Which kernel family fgd_outer_step and fgd_mix use.  AUTO (default): a TMA-pipelined kernel
 * when the tensors allow it (16-byte aligned bases, ld % 4 == 0, fewer than 2^31 - 4096
 * columns, two pipeline stages fit in shared memory), else the register kernel.  Within the
 * TMA family, K = 64, every K in [17, 63] other than 32, and a dense matrix at K = 32 run the
 * mix as a tensor-core contraction (3 x TF32 split, fp32 accumulate: relative error about
 * 2^-22 instead of fp32's 2^-24; sparse and mean mixes are densified for it); K = 2, 4, 8, 16,
 * 32 with sparse or mean mixes run compile-time fp32 kernels, other K below 17 a run-time-K
 * fp32 kernel.  REGISTER / TMA force a family (TMA fails with FGD_ERR_UNSUPPORTED when not
 * eligible); TMA_FP32 is the TMA family with every contraction kept on the fp32 CUDA cores.
 * All compute the same round. */
typedef enum { FGD_PATH_AUTO = 0, FGD_PATH_REGISTER = 1, FGD_PATH_TMA = 2, FGD_PATH_TMA_FP32 = 3 } fgd_path;
int fgd_set_path(fgd_ctx* ctx, int path);
/* Synchronises `stream` and reports whether any kernel of this context abandoned a bounded
 * device-side wait since the last check: FGD_OK, or FGD_ERR_TIMEOUT (then the outputs of the
 * affected launch are invalid).  Clears the flag. */
int fgd_device_status(fgd_ctx* ctx, void* stream);
/* Number of kernels this context has launched since creation (for launch accounting). */
int64_t fgd_launch_count(const fgd_ctx* ctx);
/* Test hooks for the bounded device-side waits (no counterpart in the paper, whose failure model
 * -- missed exchanges, Sec. 1 / Sec. 5.2 -- is pure data: edge masks).  They let a test make a
 * wait of the pipelined kernels run out WITHOUT faulting or hanging the GPU, to check that the
 * kernel then records FGD_ERR_TIMEOUT, waits for its own copies, releases its tensor memory and
 * returns, and that the context stays usable:
 *   FGD_DEBUG_SPIN_LIMIT  polls after which a device-side wait gives up (0 = the default, 2^24);
 *   FGD_DEBUG_SKIP_TILE   every CTA of the TMA-pipelined kernels (fused step, tensor-core step,
 *                         tensor-core mix) announces but never issues the loads of its value-th
 *                         tile (0-based), so the wait for that tile runs out; -1 = off (default).
 *   FGD_DEBUG_GOSSIP_PATH which kernel takes a step above 16 workers: 0 = the measured choice (default);
 *                         1 / 2 = the tensor-core kernel, a fused sparse Mix1 gathered from the staged
 *                         theta_prev (1) or, above 48 workers, run as a second group of MMAs (2); 3 = the
 *                         row-gather kernel (sparse Mix2 only).  For tests and measurements that need one
 *                         kernel whatever the shape; results agree to rounding.
 * All stay set until changed.  Not for production use. */
typedef enum { FGD_DEBUG_SPIN_LIMIT = 1, FGD_DEBUG_SKIP_TILE = 2, FGD_DEBUG_GOSSIP_PATH = 3 } fgd_debug_key;
int fgd_debug_set(fgd_ctx* ctx, int key, int64_t value);
/* Measurement aid (no counterpart in the paper): the HBM traffic of fgd_outer_step without its
 * arithmetic.  Reads theta_local, theta_prev and momentum and writes theta_new and momentum in the
 * fused step's own tiles (all K rows by a few hundred columns, the same TMA stage ring), storing
 * theta_prev's values into theta_new and the momentum's own values back: on an in-place call
 * (theta_new == theta_prev) no tensor changes.  Its time on the caller's tensors is the roofline of
 * the step's ACCESS PATTERN (3 K row streams read and 2 K written concurrently), which lies below
 * a plain copy's bandwidth, the more so the larger K is.  Device [K, ld] tensors as in
 * fgd_outer_step, same aliasing rules; needs the TMA path's alignment (else FGD_ERR_UNSUPPORTED);
 * built for K = 4, 8, 16, 32, 64. */
int fgd_debug_stream_pattern(fgd_ctx* ctx, const float* theta_local, const float* theta_prev, float* momentum,
                             float* theta_new, void* stream);

/* ---- mixing operators (Sec. 3 "Gossip-based Mixing"; App. A table of (Mix1, Mix2)) ---- */
typedef enum {
  FGD_MIX_IDENTITY = 0, /* W = I ("identity": no mixing) */
  FGD_MIX_MEAN = 1,     /* W = (1/K) 1 1^T ("global all-reduce"); ignores edge_mask, since the
                           paper's all-reduce restarts until it succeeds (Sec. 5.2) */
  FGD_MIX_SPARSE = 2,   /* neighbour list + weights (+ per-round edge mask) */
  FGD_MIX_DENSE = 3     /* explicit K x K matrix */
} fgd_mix_kind;

/* What happens to the weights when edge_mask drops an edge (the paper only says a missed
 * exchange gives weaker mixing; these rules are this library's):
 *  NONE        dropped edges get weight 0, nothing else changes (rows may sum to < 1);
 *  SELF_ABSORB surviving edges keep their base weight, both endpoints of a dropped edge add
 *              its base weight to their self weight;
 *  METROPOLIS  with d'_m = surviving degree, each surviving edge {m,n} gets
 *              1/(1+max(d'_m,d'_n)) and the self weight is 1 - (row's edge weights).
 * The last two keep W symmetric and doubly stochastic. */
typedef enum { FGD_RENORM_NONE = 0, FGD_RENORM_SELF_ABSORB = 1, FGD_RENORM_METROPOLIS = 2 } fgd_renorm;

typedef struct {
  int32_t kind;             /* fgd_mix_kind */
  int32_t K;                /* must equal the context's K */
  int32_t D;                /* SPARSE: neighbour slots per row, 0..FGD_MAX_D */
  int32_t renorm;           /* fgd_renorm, SPARSE with edge_mask */
  const int32_t* nbr;       /* SPARSE: [K*D], neighbour of worker m in slot j, -1 = empty.
                               No self loops, no duplicates in a row, symmetric (n in row m
                               iff m in row n). */
  const float* w;           /* SPARSE: [K*D] base edge weights (ignored by METROPOLIS) */
  const float* w_self;      /* SPARSE: [K] base self weights */
  const uint8_t* edge_mask; /* SPARSE: [K*D], 1 = alive, 0 = dropped; NULL = all alive.
                               Must be symmetric. */
  const float* W;           /* DENSE: [K*K] row-major, W[m*K+n] = weight worker m gives n */
} fgd_mix_desc;

/* g = theta_prev - theta_local, the negated outer pseudo-gradient Delta_m = y_{m,r,H} -
 * y_{m,r,0} (Sec. 4.1; Algorithm 1, the "outer pseudo-gradient" line; the sign is the one
 * OuterOpt receives).  g: [K, ld], may alias neither input. */
int fgd_outer_grad(fgd_ctx* ctx, const float* theta_prev, const float* theta_local, float* g,
                   void* stream);

/* out_m = sum_n W[m][n] in_n (Sec. 3, definition of Mix_W), used for Mix1 or any stand-alone
 * mix.  in: [K, ld].  out: [K, ld] (out == in allowed: in place), or, when out_is_vector != 0
 * (kind must be FGD_MIX_MEAN), the single averaged row [P]. */
int fgd_mix(fgd_ctx* ctx, const fgd_mix_desc* desc, const float* in, float* out,
            int out_is_vector, void* stream);

/* The fused outer step: outer gradient, Mix2, Nesterov update and (optionally) the consensus
 * partial sums in ONE pass over HBM (reads theta_local, theta_prev, momentum once, writes
 * theta_new, momentum once).  Sec. 4.1 last three round equations + App. B update.
 *   mix2        Mix2 applied to the outer gradient (any kind).
 *   mix1_fused  if non-NULL, Mix1 is ALSO computed in the kernel from theta_prev (kind
 *               IDENTITY, MEAN or SPARSE) and `x` must be NULL; if NULL, `x` holds the Mix1
 *               result computed earlier (e.g. by fgd_mix on a side stream): [P] when
 *               x_is_vector != 0 (the global average), else [K, ld].
 *   momentum    [K, ld], updated in place.
 *   theta_new   [K, ld]; may be exactly theta_prev (in place).  No other overlap allowed.
 *   lr, mu      outer learning rate gamma and momentum mu (used as fp32 in the kernel).
 *   cd_sumsq    NULL, or device [K] doubles receiving s_m of theta_new (see
 *               fgd_consensus_distance). */
int fgd_outer_step(fgd_ctx* ctx, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused,
                   const float* x, int x_is_vector, const float* theta_local,
                   const float* theta_prev, float* momentum, float* theta_new, double lr,
                   double mu, double* cd_sumsq, void* stream);

/* The two variants the paper adds to Algorithm 1, as options of the same fused step.
 *   mix2_ranges / n_ranges  the "-subset" configurations (Sec. 4.1, App. A): Mix2 is applied only
 *       to columns p with lo <= p < hi for one of the n_ranges (<= FGD_MAX_RANGES) host pairs
 *       {lo, hi} in mix2_ranges[2*n_ranges]; every other column passes through identity.
 *       Bounds must be multiples of 4 columns (hi may also be P).  n_ranges = 0: every column.
 *   average_momentum        the GlobalM1S configurations (App. B): Mix1 also averages the outer
 *       optimizer state, v_m <- (1/K) sum_n v_n, before the Nesterov update.  Needs Mix1 to be
 *       the global average (x given as the averaged row, or mix1_fused of kind MEAN), else
 *       FGD_ERR_UNSUPPORTED.
 *   x_next                  device [P] or NULL.  When Mix1 is the global average, next round's
 *       Mix1 result x_{r+1} = (1/K) sum_m theta_new_m depends only on this step's output, and
 *       the step already forms that column mean for the consensus term: with x_next the kernel
 *       writes it out (4/K bytes per worker-parameter more), so the caller can skip the
 *       separate fgd_mix of the next round.  Same value as launching Mix1 at the top of the
 *       next round (Algorithm 1): nothing stale.  Must not overlap any other tensor, in
 *       particular not the `x` this call reads.
 * opts == NULL is fgd_outer_step. */
typedef struct {
  const int64_t* mix2_ranges;
  int32_t n_ranges;
  int32_t average_momentum;
  float* x_next;
} fgd_step_options;
int fgd_outer_step_ex(fgd_ctx* ctx, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused,
                      const float* x, int x_is_vector, const float* theta_local,
                      const float* theta_prev, float* momentum, float* theta_new, double lr,
                      double mu, double* cd_sumsq, const fgd_step_options* opts, void* stream);

/* The same outer step (Algorithm 1, the blocking part of the round) when the inner steps'
 * result arrives from HOST memory: theta_local_host is a HOST [K, ld] matrix (pinned memory
 * for full copy bandwidth; pageable works, more slowly), theta_local_dev a DEVICE [K, ld]
 * staging matrix of the caller.  The columns are cut into n_chunks (1..FGD_MAX_CHUNKS) chunks
 * on 1024-column boundaries; chunk i+1 is copied on an internal stream while the fused step
 * of chunk i runs on `stream` (columns are independent, so the result is that of
 * fgd_outer_step on the whole matrix, bit for bit in theta_new and momentum).  cd_sumsq_host:
 * HOST [K] doubles or NULL; the per-chunk sums are added in chunk order.  No mix2_ranges /
 * momentum averaging here.  Unlike the other calls this one RETURNS AFTER THE ROUND HAS
 * COMPLETED on the device when cd_sumsq_host is given (it has to read the sums back);
 * with NULL it is asynchronous like the rest.  Only the K consensus doubles come back to the
 * host: theta_new and the momentum stay on the device, where the next round reads them.  The
 * first call creates the internal stream, events and 32 KB of device and pinned host memory (so:
 * not inside a stream capture); if that set-up fails the call returns FGD_ERR_CUDA before any
 * launch and the next call tries again.  While the call runs it narrows the context's column
 * count to the chunk it is launching: no other thread may use this context meanwhile. */
int fgd_outer_step_from_host(fgd_ctx* ctx, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused,
                             const float* x, int x_is_vector, const float* theta_local_host,
                             float* theta_local_dev, const float* theta_prev, float* momentum,
                             float* theta_new, double lr, double mu, double* cd_sumsq_host,
                             int n_chunks, void* stream);

/* s_m = sum_p (theta[m][p] - (1/K) sum_n theta[n][p])^2 into device cd_sumsq[K] (doubles).
 * The paper gives two L2 consensus distances, both functions of s: the mean of the
 * un-squared norms (Sec. 4.4) and the mean of the squared norms (App. D); see
 * fgd_cd_finalize. */
int fgd_consensus_distance(fgd_ctx* ctx, const float* theta, double* cd_sumsq, void* stream);

/* JS functional disagreement (App. D.2): for every token position u the normalised
 * Jensen-Shannon distance sqrt(JS / ln 2) between worker m's softmax distribution and the
 * parameter-averaged model's, computed in float64 in the log domain on the top_k tokens of the
 * averaged model only (the paper uses 100; both distributions are restricted to those tokens
 * and renormalised; ties at the cut go to the lower token index).  CD_JS is the mean of d_js.
 *   worker_logits device [K, U, V] fp32, avg_logits device [U, V] fp32 (the model forward that
 *   produces them is not part of this library);
 *   top_idx  device [U, top_k] int32 out: the selected tokens of each position, ascending;
 *   d_js     device [K, U] doubles out;  cd_worker device [K] doubles out: mean over u.
 * 1 <= top_k <= min(256, V).  Needs no context and allocates nothing. */
int fgd_js_distance(int device, int K, int64_t U, int64_t V, int top_k, const float* worker_logits,
                    const float* avg_logits, int32_t* top_idx, double* d_js, double* cd_worker,
                    void* stream);

/* (No counterpart in the paper: a packaging variant of fgd_consensus_distance.)
 * Same result as fgd_consensus_distance, for callers that cannot allocate GPU memory and so
 * cannot create a context: it needs no fgd_ctx and calls no cudaMalloc / cudaFree or any other
 * allocating routine.  Its per-CTA partial sums live in a fixed 512 KiB device array that is
 * part of the library image (1024 CTAs x FGD_MAX_K workers x 8 bytes), resident on every GPU
 * that loads the library until the process exits.
 *   device, K, P, ld   as in fgd_create; K > FGD_MAX_K does not fit the array and is rejected
 *                      with FGD_ERR_INVALID_ARG (any P is fine: the grid is capped at 1024 CTAs).
 *   theta              device [K, ld] fp32; cd_sumsq device [K] doubles (caller-owned).
 * The first call on a device resolves the array's device address (once per device); make that
 * first call before starting any stream capture.  All calls share the one array and it keeps
 * the previous call's contents (nothing in it needs to start at zero): two calls that overlap
 * on the same GPU race and return wrong sums, so order them on one stream or with events.
 * Errors: reason via fgd_last_error(NULL). */
int fgd_consensus_distance_noalloc(int device, int K, int64_t P, int64_t ld, const float* theta,
                                   double* cd_sumsq, void* stream);

/* ---------------------------- host helpers (pure CPU) ---------------------------------- */
/* Topologies.  Each writes nbr[K*D], w[K*D], w_self[K] for the D it documents and returns D
 * (>= 0) or a negative status.  Weights are Metropolis weights of the unmasked graph.
 *  ring:            D = 2, slots (m-1) mod K, (m+1) mod K; K == 2 uses slot 0 only; 1/3 each.
 *  onepeer_xor:     D = 1, partner m XOR 2^(round mod log2 K), weight 1/2; K a power of two.
 *  hypercube:       D = log2 K, slot j = m XOR 2^j, weights 1/(1 + log2 K); K a power of two.
 *  random_matching: D = 1, one random perfect matching per (seed, round, mix_id), each pair
 *                   averages (the paper's "pairwise gossip", Sec. 3); odd K leaves one idle. */
int fgd_topo_ring(int K, int32_t* nbr, float* w, float* w_self);
int fgd_topo_onepeer_xor(int K, int64_t round, int32_t* nbr, float* w, float* w_self);
int fgd_topo_hypercube(int K, int32_t* nbr, float* w, float* w_self);
int fgd_topo_random_matching(int K, uint64_t seed, int64_t round, int mix_id, int32_t* nbr,
                             float* w, float* w_self);
/* Transient link failures (Sec. 1, Sec. 5.2): every undirected edge is dropped independently
 * with probability p_fail in round `round`; mix_id (1 = Mix1, 2 = Mix2) gives the two
 * transfers of a round independent draws.  Counter-based and order independent: edge {a,b}
 * is dropped iff the top 32 bits of H(seed, round, mix_id, min, max) are below
 * floor(p_fail * 2^32).  mask_out[K*D]: 1 alive, 0 dropped or empty slot. */
int fgd_edge_mask(uint64_t seed, int64_t round, int mix_id, double p_fail, int K, int D,
                  const int32_t* nbr, uint8_t* mask_out);
/* The 64-bit hash behind fgd_edge_mask and fgd_topo_random_matching (exposed for tests). */
uint64_t fgd_hash64(uint64_t seed, uint64_t round, uint64_t tag, uint64_t a, uint64_t b);
/* Effective weights of a SPARSE descriptor after mask + renormalisation:
 * w_eff[K*D], w_self_eff[K] (doubles).  Also validates the descriptor. */
int fgd_effective_weights(const fgd_mix_desc* desc, double* w_eff, double* w_self_eff);
/* Dense K x K row-convention matrix of any descriptor (doubles, row-major). */
int fgd_dense_matrix(const fgd_mix_desc* desc, double* W_out);
/* From s[K] (host doubles): *cd_mean_norm = (1/K) sum sqrt(s_m)  (Sec. 4.4),
 *                           *cd_mean_sq   = (1/K) sum s_m         (App. D). */
int fgd_cd_finalize(const double* sumsq_host, int K, double* cd_mean_norm, double* cd_mean_sq);

#ifdef __cplusplus
}
#endif
#endif /* FGD_H_ */
