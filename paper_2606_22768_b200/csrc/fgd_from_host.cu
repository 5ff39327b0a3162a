// fgd_outer_step_from_host: the fused outer step fed from host memory, column chunk by column
// chunk, with the host-to-device copy of the next chunk overlapping the step of the current one.
#include <cuda_runtime.h>

#include "../../include/fgd.h"
#include "fgd_ctx.h"
#include "fgd_nvtx.h"

namespace {

// Frees whatever the streaming set-up has created so far and leaves every handle null.
void release_streaming_resources(fgd_ctx* c) {
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->start_ev) cudaEventDestroy(c->start_ev);
  for (cudaEvent_t& ev : c->chunk_ev) {
    if (ev) cudaEventDestroy(ev);
    ev = nullptr;
  }
  if (c->chunk_cd) cudaFree(c->chunk_cd);
  if (c->chunk_cd_host) cudaFreeHost(c->chunk_cd_host);
  c->copy_stream = nullptr;
  c->start_ev = nullptr;
  c->chunk_cd = nullptr;
  c->chunk_cd_host = nullptr;
  c->streaming_ready = false;
}

// Creates the copy stream, the events and the two small consensus buffers.  All or nothing: when
// any step fails everything made so far is released again, so a later call starts from scratch
// instead of running with a missing buffer.
int ensure_streaming_resources(fgd_ctx* c) {
  if (c->streaming_ready) return FGD_OK;
  cudaError_t e = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->start_ev, cudaEventDisableTiming);
  for (int i = 0; i < FGD_MAX_CHUNKS && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&c->chunk_ev[i], cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMalloc(&c->chunk_cd, sizeof(double) * FGD_MAX_CHUNKS * FGD_MAX_K);
  if (e == cudaSuccess) e = cudaMallocHost(&c->chunk_cd_host, sizeof(double) * FGD_MAX_CHUNKS * FGD_MAX_K);
  if (e != cudaSuccess || !c->copy_stream || !c->start_ev || !c->chunk_cd || !c->chunk_cd_host) {
    release_streaming_resources(c);
    cudaGetLastError();
    return fail(c, FGD_ERR_CUDA, "fgd_outer_step_from_host: set-up of the copy stream and buffers failed: %s",
                e != cudaSuccess ? cudaGetErrorString(e) : "a handle is missing");
  }
  c->streaming_ready = true;
  return FGD_OK;
}

// The step of one column window runs through the ordinary entry point with the context's column
// count narrowed to the window (same row stride); restored on every exit path.  This is why a
// context must not be shared between threads while this call runs.
struct ColumnWindow {
  fgd_ctx* c;
  int64_t saved;
  ColumnWindow(fgd_ctx* ctx, int64_t cols) : c(ctx), saved(ctx->P) { c->P = cols; }
  ~ColumnWindow() { c->P = saved; }
};

}  // namespace

extern "C" int fgd_outer_step_from_host(fgd_ctx* c, const fgd_mix_desc* mix2, const fgd_mix_desc* mix1_fused,
                                        const float* x, int x_is_vector, const float* theta_local_host,
                                        float* theta_local_dev, const float* theta_prev, float* momentum,
                                        float* theta_new, double lr, double mu, double* cd_sumsq_host,
                                        int n_chunks, void* stream) {
  FGD_NVTX_RANGE("fgd_outer_step_from_host");
  if (!c) return fail(nullptr, FGD_ERR_INVALID_ARG, "fgd_outer_step_from_host: ctx is NULL");
  if (!theta_local_host || !theta_local_dev || !theta_prev || !momentum || !theta_new)
    return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step_from_host: NULL tensor");
  if (n_chunks < 1 || n_chunks > FGD_MAX_CHUNKS)
    return fail(c, FGD_ERR_INVALID_ARG, "fgd_outer_step_from_host: n_chunks %d not in [1, %d]", n_chunks, FGD_MAX_CHUNKS);
  DeviceGuard guard(c->device);
  if (!guard.ok) return fail(c, FGD_ERR_CUDA, "cannot select device %d", c->device);
  if (int rc = ensure_streaming_resources(c)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int K = c->K;
  const int64_t P = c->P, ld = c->ld;
  // chunk width: whole 1024-column blocks (tile and vector boundaries of every kernel)
  int64_t w = (P + n_chunks - 1) / n_chunks;
  w = (w + 1023) / 1024 * 1024;
  const int n = (int)((P + w - 1) / w);

  // the staging matrix may still be read by earlier work on `stream`
  FGD_CUDA(c, cudaEventRecord(c->start_ev, st));
  FGD_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->start_ev, 0));
  for (int i = 0; i < n; ++i) {
    const int64_t c0 = (int64_t)i * w, c1 = c0 + w < P ? c0 + w : P;
    FGD_CUDA(c, cudaMemcpy2DAsync(theta_local_dev + c0, sizeof(float) * (size_t)ld, theta_local_host + c0,
                                  sizeof(float) * (size_t)ld, sizeof(float) * (size_t)(c1 - c0), (size_t)K,
                                  cudaMemcpyHostToDevice, c->copy_stream));
    FGD_CUDA(c, cudaEventRecord(c->chunk_ev[i], c->copy_stream));
  }
  int rc = FGD_OK;
  for (int i = 0; i < n && rc == FGD_OK; ++i) {
    const int64_t c0 = (int64_t)i * w, c1 = c0 + w < P ? c0 + w : P;
    FGD_CUDA(c, cudaStreamWaitEvent(st, c->chunk_ev[i], 0));
    ColumnWindow window(c, c1 - c0);   // the window [c0, c1) of every matrix: same row stride, fewer columns
    rc = fgd_outer_step_ex(c, mix2, mix1_fused, x ? x + c0 : nullptr, x_is_vector, theta_local_dev + c0, theta_prev + c0,
                           momentum + c0, theta_new + c0, lr, mu, cd_sumsq_host ? c->chunk_cd + (size_t)i * K : nullptr,
                           nullptr, st);
  }
  if (rc != FGD_OK) return rc;
  if (cd_sumsq_host) {
    FGD_CUDA(c, cudaMemcpyAsync(c->chunk_cd_host, c->chunk_cd, sizeof(double) * (size_t)n * K, cudaMemcpyDeviceToHost, st));
    FGD_CUDA(c, cudaStreamSynchronize(st));
    for (int m = 0; m < K; ++m) {
      double s = 0.0;
      for (int i = 0; i < n; ++i) s += c->chunk_cd_host[(size_t)i * K + m];
      cd_sumsq_host[m] = s;
    }
  }
  return FGD_OK;
}
