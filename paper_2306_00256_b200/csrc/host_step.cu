// Host-memory front end of the fused step, and the workspace size query.
//
// The update mixes rows only, never columns, so a column slab of all n rows is a complete
// sub-problem.  The host variant streams slabs through the device: while slab j is being
// updated, slab j+1 is on its way in and slab j-1 on its way out (three buffer sets, one
// stream each; the copy engines run host->device and device->host transfers concurrently).
#include <cuda_runtime.h>

#include <cstdint>

#include "ceca.h"
#include "plan.h"

namespace ceca {

cudaError_t enqueue_step(const Plan &plan, const float *X, const float *Y, const float *G, float *Xo,
                         float *Yo, int32_t n, int64_t d, int64_t ld, float gamma,
                         cudaStream_t stream);
size_t logreg_workspace_bytes(int32_t n, int32_t m, int64_t d);

constexpr int kHostBuffers = 3;
constexpr int64_t kHostMinSlabCols = 4;

static inline size_t host_slab_bytes(int32_t n, int64_t cols) { return (size_t)3 * n * cols * sizeof(float); }

}  // namespace ceca

extern "C" size_t ceca_workspace_bytes(ceca_workspace_kind_t kind, int32_t n, int32_t m, int64_t d) {
  using namespace ceca;
  if (n < 1 || d < 1) return 0;
  switch (kind) {
    case CECA_WS_CONSENSUS_FUSED: return 256;
    case CECA_WS_CONSENSUS_UNFUSED: return (size_t)n * (size_t)d * sizeof(float);
    case CECA_WS_LOGREG_GRAD: return m < 1 ? 0 : logreg_workspace_bytes(n, m, d);
    case CECA_WS_STEP_HOST: return kHostBuffers * host_slab_bytes(n, kHostMinSlabCols);
  }
  return 0;
}

extern "C" ceca_status_t ceca_gossip_sgd_step_host(float *X, float *Y, const float *G, int32_t n, int64_t d,
                                                   int64_t ld, float gamma, ceca_variant_t variant, int64_t k,
                                                   void *workspace, size_t workspace_bytes) {
  using namespace ceca;
  if (!X || !Y || n < 1 || d < 1 || ld < d) return CECA_ERR_INVALID_ARG;
  Plan plan;
  ceca_status_t st = make_plan(n, variant, k, &plan);
  if (st != CECA_OK) return st;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      workspace_bytes < kHostBuffers * host_slab_bytes(n, kHostMinSlabCols))
    return CECA_ERR_WORKSPACE;

  // slab width: a multiple of 4 columns such that three buffer sets fit in the workspace,
  // narrowed to give at least eight slabs (when they stay wide) so copies and kernels overlap
  const int64_t w_fit = (int64_t)(workspace_bytes / (kHostBuffers * (size_t)3 * n * sizeof(float))) / 4 * 4;
  int64_t w = w_fit < ((d + 3) / 4) * 4 ? w_fit : ((d + 3) / 4) * 4;
  const int64_t w_eighth = (((d + 7) / 8) + 63) / 64 * 64;
  if (w_eighth >= 16384 && w_eighth < w) w = w_eighth;

  cudaStream_t streams[kHostBuffers];
  for (int b = 0; b < kHostBuffers; ++b)
    if (cudaStreamCreateWithFlags(&streams[b], cudaStreamNonBlocking) != cudaSuccess) {
      for (int c = 0; c < b; ++c) cudaStreamDestroy(streams[c]);
      return CECA_ERR_CUDA;
    }

  cudaError_t err = cudaSuccess;
  const size_t pitch = (size_t)w * sizeof(float);
  int64_t slab = 0;
  for (int64_t c0 = 0; c0 < d && err == cudaSuccess; c0 += w, ++slab) {
    const int b = (int)(slab % kHostBuffers);
    cudaStream_t s = streams[b];
    float *dx = reinterpret_cast<float *>(static_cast<char *>(workspace) + (size_t)b * host_slab_bytes(n, w));
    float *dy = dx + (size_t)n * w;
    float *dg = dy + (size_t)n * w;
    const int64_t cols = (d - c0 < w) ? d - c0 : w;
    const size_t width = (size_t)cols * sizeof(float);
    const size_t hpitch = (size_t)ld * sizeof(float);
    err = cudaMemcpy2DAsync(dx, pitch, X + c0, hpitch, width, n, cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess && plan.reads_y)
      err = cudaMemcpy2DAsync(dy, pitch, Y + c0, hpitch, width, n, cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess && G)
      err = cudaMemcpy2DAsync(dg, pitch, G + c0, hpitch, width, n, cudaMemcpyHostToDevice, s);
    if (err == cudaSuccess)
      err = enqueue_step(plan, dx, plan.reads_y ? dy : nullptr, G ? dg : nullptr, dx, dy, n, cols, w, gamma, s);
    if (err == cudaSuccess)
      err = cudaMemcpy2DAsync(X + c0, hpitch, dx, pitch, width, n, cudaMemcpyDeviceToHost, s);
    if (err == cudaSuccess)
      err = cudaMemcpy2DAsync(Y + c0, hpitch, dy, pitch, width, n, cudaMemcpyDeviceToHost, s);
  }
  for (int b = 0; b < kHostBuffers; ++b) {
    cudaError_t e = cudaStreamSynchronize(streams[b]);
    if (err == cudaSuccess) err = e;
    cudaStreamDestroy(streams[b]);
  }
  return err == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}
