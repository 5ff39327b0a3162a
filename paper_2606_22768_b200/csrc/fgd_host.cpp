// Host-side (pure CPU) parts of the library: topology builders, per-round edge-failure
// masks, weight renormalisation, descriptor validation, consensus-distance finalisation.
// Everything here is integer / double arithmetic on tiny arrays (K <= 64, D <= 8).
#include <cmath>
#include <cstdio>
#include <cstring>

#include "fgd_internal.h"

namespace fgd {

thread_local char g_thread_error[256] = "";

void set_thread_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_thread_error, sizeof(g_thread_error), fmt, ap);
  va_end(ap);
}

// splitmix64 output function.
static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

static const uint64_t kGolden = 0x9E3779B97F4A7C15ull;
static const uint64_t kTagMatching = 16;

uint64_t hash64(uint64_t seed, uint64_t round, uint64_t tag, uint64_t a, uint64_t b) {
  uint64_t h = mix64(seed + kGolden);
  const uint64_t words[4] = {round, tag, a, b};
  for (int i = 0; i < 4; ++i) h = mix64((h ^ words[i]) + kGolden);
  return h;
}

static bool is_pow2(int k) { return k >= 1 && (k & (k - 1)) == 0; }
static int ilog2(int k) {
  int b = 0;
  while ((1 << (b + 1)) <= k) ++b;
  return b;
}

static int check_K(int K) {
  if (K < 1 || K > FGD_MAX_K) {
    set_thread_error("K=%d out of range [1, %d]", K, FGD_MAX_K);
    return FGD_ERR_INVALID_ARG;
  }
  return FGD_OK;
}

// Validates a descriptor against K; on failure writes the reason into msg.
int validate_desc(const fgd_mix_desc* d, int K, char* msg, size_t msg_len) {
#define FAIL(...)                          \
  do {                                     \
    snprintf(msg, msg_len, __VA_ARGS__);   \
    return FGD_ERR_INVALID_ARG;            \
  } while (0)
  if (!d) FAIL("mix descriptor is NULL");
  if (d->K != K) FAIL("descriptor K=%d does not match K=%d", d->K, K);
  if (K < 1 || K > FGD_MAX_K) FAIL("K=%d out of range [1, %d]", K, FGD_MAX_K);
  switch (d->kind) {
    case FGD_MIX_IDENTITY:
    case FGD_MIX_MEAN:
      return FGD_OK;
    case FGD_MIX_DENSE:
      if (!d->W) FAIL("dense mix needs W");
      for (int i = 0; i < K * K; ++i)
        if (!std::isfinite(d->W[i])) FAIL("dense W[%d] is not finite", i);
      return FGD_OK;
    case FGD_MIX_SPARSE:
      break;
    default:
      FAIL("unknown mix kind %d", d->kind);
  }
  if (d->D < 0 || d->D > FGD_MAX_D) FAIL("D=%d out of range [0, %d]", d->D, FGD_MAX_D);
  if (d->renorm < FGD_RENORM_NONE || d->renorm > FGD_RENORM_METROPOLIS)
    FAIL("unknown renorm rule %d", d->renorm);
  if (!d->w_self) FAIL("sparse mix needs w_self");
  if (d->D > 0 && (!d->nbr || !d->w)) FAIL("sparse mix with D>0 needs nbr and w");
  const int D = d->D;
  for (int m = 0; m < K; ++m) {
    if (!std::isfinite(d->w_self[m])) FAIL("w_self[%d] is not finite", m);
    for (int j = 0; j < D; ++j) {
      const int n = d->nbr[m * D + j];
      if (n == -1) continue;
      if (n < 0 || n >= K) FAIL("nbr[%d][%d]=%d out of range", m, j, n);
      if (n == m) FAIL("nbr[%d][%d] is a self loop", m, j);
      if (!std::isfinite(d->w[m * D + j])) FAIL("w[%d][%d] is not finite", m, j);
      for (int i = 0; i < j; ++i)
        if (d->nbr[m * D + i] == n) FAIL("worker %d lists neighbour %d twice", m, n);
    }
  }
  for (int m = 0; m < K; ++m) {
    for (int j = 0; j < D; ++j) {
      const int n = d->nbr[m * D + j];
      if (n == -1) continue;
      int back = -1;
      for (int i = 0; i < D; ++i)
        if (d->nbr[n * D + i] == m) back = i;
      if (back < 0) FAIL("edge %d->%d has no reverse edge", m, n);
      if (d->edge_mask && (d->edge_mask[m * D + j] != 0) != (d->edge_mask[n * D + back] != 0))
        FAIL("edge_mask is not symmetric on edge {%d,%d}", m, n);
    }
  }
  return FGD_OK;
#undef FAIL
}

// Effective weights after mask + renormalisation (doubles).  Descriptor already validated.
void effective_weights(const fgd_mix_desc* d, double* w_eff, double* ws_eff) {
  const int K = d->K, D = d->D;
  bool alive[FGD_MAX_K * FGD_MAX_D];
  int deg[FGD_MAX_K];
  for (int m = 0; m < K; ++m) {
    deg[m] = 0;
    for (int j = 0; j < D; ++j) {
      const bool a = d->nbr[m * D + j] >= 0 && (!d->edge_mask || d->edge_mask[m * D + j] != 0);
      alive[m * D + j] = a;
      deg[m] += a ? 1 : 0;
    }
  }
  for (int m = 0; m < K; ++m) {
    if (d->renorm == FGD_RENORM_METROPOLIS) {
      double tot = 0.0;
      for (int j = 0; j < D; ++j) {
        double wt = 0.0;
        if (alive[m * D + j]) {
          const int n = d->nbr[m * D + j];
          wt = 1.0 / (1.0 + (double)(deg[m] > deg[n] ? deg[m] : deg[n]));
          tot += wt;
        }
        w_eff[m * D + j] = wt;
      }
      ws_eff[m] = 1.0 - tot;
    } else {
      double ws = (double)d->w_self[m];
      for (int j = 0; j < D; ++j) {
        double wt = 0.0;
        if (alive[m * D + j]) {
          wt = (double)d->w[m * D + j];
        } else if (d->nbr[m * D + j] >= 0 && d->renorm == FGD_RENORM_SELF_ABSORB) {
          ws += (double)d->w[m * D + j];
        }
        w_eff[m * D + j] = wt;
      }
      ws_eff[m] = ws;
    }
  }
}

}  // namespace fgd

using namespace fgd;

extern "C" {

uint64_t fgd_hash64(uint64_t seed, uint64_t round, uint64_t tag, uint64_t a, uint64_t b) {
  return hash64(seed, round, tag, a, b);
}

int fgd_topo_ring(int K, int32_t* nbr, float* w, float* w_self) {
  if (int rc = check_K(K)) return rc;
  if (!nbr || !w || !w_self) {
    set_thread_error("fgd_topo_ring: NULL output");
    return FGD_ERR_INVALID_ARG;
  }
  for (int m = 0; m < K; ++m) {
    if (K == 1) {
      nbr[2 * m] = nbr[2 * m + 1] = -1;
      w[2 * m] = w[2 * m + 1] = 0.f;
      w_self[m] = 1.f;
    } else if (K == 2) {
      nbr[2 * m] = 1 - m;
      nbr[2 * m + 1] = -1;
      w[2 * m] = 0.5f;
      w[2 * m + 1] = 0.f;
      w_self[m] = 0.5f;
    } else {
      nbr[2 * m] = (m + K - 1) % K;
      nbr[2 * m + 1] = (m + 1) % K;
      w[2 * m] = w[2 * m + 1] = (float)(1.0 / 3.0);
      w_self[m] = (float)(1.0 / 3.0);
    }
  }
  return 2;
}

int fgd_topo_onepeer_xor(int K, int64_t round, int32_t* nbr, float* w, float* w_self) {
  if (int rc = check_K(K)) return rc;
  if (!is_pow2(K) || round < 0 || !nbr || !w || !w_self) {
    set_thread_error("fgd_topo_onepeer_xor: K=%d must be a power of two, round >= 0, outputs non-NULL", K);
    return FGD_ERR_INVALID_ARG;
  }
  const int bits = ilog2(K);
  for (int m = 0; m < K; ++m) {
    if (bits == 0) {
      nbr[m] = -1;
      w[m] = 0.f;
      w_self[m] = 1.f;
    } else {
      nbr[m] = m ^ (1 << (int)(round % bits));
      w[m] = 0.5f;
      w_self[m] = 0.5f;
    }
  }
  return 1;
}

int fgd_topo_hypercube(int K, int32_t* nbr, float* w, float* w_self) {
  if (int rc = check_K(K)) return rc;
  if (!is_pow2(K) || !nbr || !w || !w_self) {
    set_thread_error("fgd_topo_hypercube: K=%d must be a power of two, outputs non-NULL", K);
    return FGD_ERR_INVALID_ARG;
  }
  const int bits = ilog2(K);
  if (bits == 0) {
    nbr[0] = -1;
    w[0] = 0.f;
    w_self[0] = 1.f;
    return 1;
  }
  const float wt = (float)(1.0 / (1.0 + bits));
  for (int m = 0; m < K; ++m) {
    for (int j = 0; j < bits; ++j) {
      nbr[m * bits + j] = m ^ (1 << j);
      w[m * bits + j] = wt;
    }
    w_self[m] = wt;
  }
  return bits;
}

int fgd_topo_random_matching(int K, uint64_t seed, int64_t round, int mix_id, int32_t* nbr,
                             float* w, float* w_self) {
  if (int rc = check_K(K)) return rc;
  if (round < 0 || !nbr || !w || !w_self) {
    set_thread_error("fgd_topo_random_matching: round >= 0 and non-NULL outputs required");
    return FGD_ERR_INVALID_ARG;
  }
  int pi[FGD_MAX_K];
  for (int i = 0; i < K; ++i) pi[i] = i;
  for (int i = K - 1; i >= 1; --i) {
    const int j = (int)(hash64(seed, (uint64_t)round, kTagMatching + (uint64_t)mix_id, (uint64_t)i, 0) %
                        (uint64_t)(i + 1));
    const int t = pi[i];
    pi[i] = pi[j];
    pi[j] = t;
  }
  for (int m = 0; m < K; ++m) {
    nbr[m] = -1;
    w[m] = 0.f;
    w_self[m] = 1.f;
  }
  for (int t = 0; t + 1 < K; t += 2) {
    const int a = pi[t], b = pi[t + 1];
    nbr[a] = b;
    nbr[b] = a;
    w[a] = w[b] = 0.5f;
    w_self[a] = w_self[b] = 0.5f;
  }
  return 1;
}

int fgd_edge_mask(uint64_t seed, int64_t round, int mix_id, double p_fail, int K, int D,
                  const int32_t* nbr, uint8_t* mask_out) {
  if (int rc = check_K(K)) return rc;
  if (D < 0 || D > FGD_MAX_D || round < 0 || !(p_fail == p_fail) || (D > 0 && (!nbr || !mask_out))) {
    set_thread_error("fgd_edge_mask: bad D=%d, round, p_fail or NULL pointer", D);
    return FGD_ERR_INVALID_ARG;
  }
  uint64_t T;
  if (p_fail <= 0.0) T = 0;
  else if (p_fail >= 1.0) T = 1ull << 32;
  else T = (uint64_t)std::floor(p_fail * 4294967296.0);
  for (int m = 0; m < K; ++m)
    for (int j = 0; j < D; ++j) {
      const int n = nbr[m * D + j];
      if (n < 0) {
        mask_out[m * D + j] = 0;
        continue;
      }
      if (n >= K || n == m) {
        set_thread_error("fgd_edge_mask: nbr[%d][%d]=%d invalid", m, j, n);
        return FGD_ERR_INVALID_ARG;
      }
      const uint64_t lo = m < n ? m : n, hi = m < n ? n : m;
      const uint64_t h = hash64(seed, (uint64_t)round, (uint64_t)mix_id, lo, hi);
      mask_out[m * D + j] = ((h >> 32) < T) ? 0 : 1;
    }
  return FGD_OK;
}

int fgd_effective_weights(const fgd_mix_desc* desc, double* w_eff, double* w_self_eff) {
  if (!desc || desc->kind != FGD_MIX_SPARSE || !w_self_eff || (desc->D > 0 && !w_eff)) {
    set_thread_error("fgd_effective_weights: needs a SPARSE descriptor and output arrays");
    return FGD_ERR_INVALID_ARG;
  }
  if (int rc = validate_desc(desc, desc->K, g_thread_error, sizeof(g_thread_error))) return rc;
  effective_weights(desc, w_eff, w_self_eff);
  return FGD_OK;
}

int fgd_dense_matrix(const fgd_mix_desc* desc, double* W_out) {
  if (!desc || !W_out) {
    set_thread_error("fgd_dense_matrix: NULL argument");
    return FGD_ERR_INVALID_ARG;
  }
  const int K = desc->K;
  if (int rc = validate_desc(desc, K, g_thread_error, sizeof(g_thread_error))) return rc;
  for (int i = 0; i < K * K; ++i) W_out[i] = 0.0;
  switch (desc->kind) {
    case FGD_MIX_IDENTITY:
      for (int m = 0; m < K; ++m) W_out[m * K + m] = 1.0;
      break;
    case FGD_MIX_MEAN:
      for (int i = 0; i < K * K; ++i) W_out[i] = 1.0 / (double)K;
      break;
    case FGD_MIX_DENSE:
      for (int i = 0; i < K * K; ++i) W_out[i] = (double)desc->W[i];
      break;
    default: {
      double w_eff[FGD_MAX_K * FGD_MAX_D], ws_eff[FGD_MAX_K];
      effective_weights(desc, w_eff, ws_eff);
      for (int m = 0; m < K; ++m) {
        W_out[m * K + m] += ws_eff[m];
        for (int j = 0; j < desc->D; ++j) {
          const int n = desc->nbr[m * desc->D + j];
          if (n >= 0) W_out[m * K + n] += w_eff[m * desc->D + j];
        }
      }
    }
  }
  return FGD_OK;
}

int fgd_cd_finalize(const double* s, int K, double* cd_mean_norm, double* cd_mean_sq) {
  if (!s || K < 1 || K > FGD_MAX_K || !cd_mean_norm || !cd_mean_sq) {
    set_thread_error("fgd_cd_finalize: bad argument");
    return FGD_ERR_INVALID_ARG;
  }
  double a = 0.0, b = 0.0;
  for (int m = 0; m < K; ++m) {
    const double sm = s[m] > 0.0 ? s[m] : 0.0;
    a += std::sqrt(sm);
    b += sm;
  }
  *cd_mean_norm = a / K;
  *cd_mean_sq = b / K;
  return FGD_OK;
}

const char* fgd_status_string(int status) {
  switch (status) {
    case FGD_OK: return "ok";
    case FGD_ERR_INVALID_ARG: return "invalid argument";
    case FGD_ERR_ALIGNMENT: return "alignment";
    case FGD_ERR_ALIAS: return "forbidden aliasing";
    case FGD_ERR_UNSUPPORTED: return "unsupported";
    case FGD_ERR_CUDA: return "CUDA error";
    case FGD_ERR_TIMEOUT: return "device wait timed out";
    default: return "unknown status";
  }
}

}  // extern "C"
