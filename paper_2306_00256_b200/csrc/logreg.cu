// Per-agent gradients e^(k) of Algorithm 1 for two data-fitting losses over local samples (a_s, t_s):
//   logistic (synthetic classification workloads; this loss is not from the paper)
//     G[i, :] = -(1/m) sum_s l_s sigma(-l_s <a_s, z_i>) a_s
//   least squares (Sec. 5 "DSGD: least-squares problem": f_i(w) = 1/2 ||A_i w - b_i||^2)
//     G[i, :] = sum_s (<a_s, z_i> - b_s) a_s  (+ eps_i, the caller's gradient noise)
// with z = X if delta_r = 1 else Y.  Both are "coefficient per sample times the sample", so they
// share the kernels below; only the coefficient differs.
//
// Main path (d a multiple of 4, d <= 65536, 16-byte aligned rows): A is read exactly once.  A CTA
// takes one agent and a block of its samples; each thread keeps its slice of z_i and of the
// running gradient in registers, loads its slice of four sample rows, the CTA reduces the four
// inner products (warp shuffles, then a fixed-order sum over the warps through shared memory),
// every thread turns them into the four coefficients and adds coefficient * row slice to its
// gradient slice.  Per-CTA partial gradients go to the workspace and a second kernel adds them in
// a fixed order, so the result does not change from run to run.  Not a dense contraction worth
// tensor cores: two matrix-vector products per agent, bound by reading A from HBM.
// A CTA's registers hold up to 8192 columns.  Wider models run the same kernel as a thread-block
// cluster of up to eight CTAs, one column chunk each: every CTA writes its share of the inner
// products into the shared memory of all CTAs of the cluster (distributed shared memory), one
// cluster barrier makes them visible, and every CTA adds the shares in rank order, so all of them
// get the same bits.
//
// Fallback: A is read twice.  Aligned rows of more than 65536 columns: inner products, coefficients, then the
// A^T pass, all with 128-bit streaming loads (the kernels of the column-sharded form).  Any other d or
// alignment: coefficients (one warp per sample), then a column-wise accumulation with scalar loads.
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "ceca.h"
#include "plan.h"

namespace ceca {

constexpr int kLrThreads = 256;      // threads per CTA; 512 for chunks wider than 4096 columns
constexpr int kLrMaxVpt = 4;         // float4 column groups per thread -> 512*4*4 = 8192 columns per CTA
constexpr int kLrMaxCluster = 8;     // CTAs (column chunks) per cluster: the portable maximum
constexpr int kLrChunkCols = 2 * kLrThreads * 4 * kLrMaxVpt;
constexpr int kLrHalfChunkCols = kLrChunkCols / 2;   // four float4 per thread: two CTAs per SM, four rows in flight
constexpr int kLrTargetCtas = 148 * 12;

// Sample rows in flight per thread.
template <int VPT> struct LrSamples { static constexpr int value = 4; };
// NS inner products travel as one vector (one shared-memory access).
template <int NS> struct LrDots;
template <> struct LrDots<4> { using type = float4; };
template <> struct LrDots<2> { using type = float2; };
__device__ __forceinline__ void dots_add(float4 &t, float4 v) { t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w; }
__device__ __forceinline__ void dots_add(float2 &t, float2 v) { t.x += v.x; t.y += v.y; }
__device__ __forceinline__ float4 dots_pack(const float (&d)[4]) { return make_float4(d[0], d[1], d[2], d[3]); }
__device__ __forceinline__ float2 dots_pack(const float (&d)[2]) { return make_float2(d[0], d[1]); }
__device__ __forceinline__ void dots_unpack(float4 v, float (&d)[4]) { d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w; }
__device__ __forceinline__ void dots_unpack(float2 v, float (&d)[2]) { d[0] = v.x; d[1] = v.y; }

// Column chunks (CTAs per cluster) for d columns.  One CTA while its registers hold the row
// (d <= 8192: a cluster barrier per batch of rows costs more than it wins, 0.66 of the copy rate
// for two CTAs of 4096 columns against 0.78 and more for one CTA at d = 8192); beyond that chunks of 4096 columns (two CTAs per SM,
// four rows in flight) while a cluster of eight covers the row, chunks of up to 8192 columns above.
static inline int32_t logreg_chunks(int64_t d) {
  if (d <= kLrChunkCols) return 1;
  const int64_t half = (d + kLrHalfChunkCols - 1) / kLrHalfChunkCols;
  return (int32_t)(half <= kLrMaxCluster ? half : (d + kLrChunkCols - 1) / kLrChunkCols);
}

static inline int32_t logreg_sample_blocks(int32_t n, int32_t m, int64_t d) {
  const int64_t ctas_per_block = (int64_t)n * logreg_chunks(d);
  int64_t p = (kLrTargetCtas + ctas_per_block - 1) / ctas_per_block;
  const int64_t most = (m + 15) / 16;  // at least 16 samples per block
  if (p > most) p = most;
  if (p < 1) p = 1;
  return (int32_t)p;
}

constexpr int kLossLogistic = 0;
constexpr int kLossSquare = 1;

// The per-sample coefficient c_s such that the gradient is sum_s c_s a_s; t = <a_s, z_i>.
template <int LOSS>
__device__ __forceinline__ float sample_coef(float target, float t, float inv_m) {
  if (LOSS == kLossLogistic) return -target * inv_m / (1.f + expf(target * t));  // -l sigma(-l t) / m
  return t - target;                                                             // residual a.z - b
}

struct LogregArgs {
  const float *A, *labels, *Z;
  float *partial;   // [n][P][d]
  int64_t d, ld;
  int64_t chunk4;   // float4 column groups per CTA of a cluster (all of them when there is one CTA)
  int32_t n, m, P, samples_per_block, chunks;
  float inv_m;
};

__device__ __forceinline__ float dot4(float4 a, float4 b) {
  return fmaf(a.x, b.x, fmaf(a.y, b.y, fmaf(a.z, b.z, a.w * b.w)));
}

// T threads, VPT float4 column groups per thread (a chunk of up to T * VPT * 4 columns; 4096 < columns
// <= 8192 take 512 threads of four groups rather than 256 of eight: the same registers per thread and
// warps per SM as two CTAs of the 4096-column shape).  CLUSTER: launched as clusters of p.chunks CTAs
// along x; the CTA of rank r takes the column groups [r * chunk4, (r + 1) * chunk4).
template <int VPT, int LOSS, bool CLUSTER, int T>
__global__ void __launch_bounds__(T, T > 256 ? 1 : VPT == 1 ? 4 : VPT == 2 ? 3 : 2)
logreg_fused_kernel(const LogregArgs p) {
  constexpr int kWarps = T / 32;
  constexpr int NS = LrSamples<VPT>::value;
  using Dots = typename LrDots<NS>::type;
  __shared__ Dots red[2][kWarps];
  __shared__ Dots share[2][kLrMaxCluster];   // the inner-product shares of the cluster's CTAs
  namespace cg = cooperative_groups;
  const int rank = CLUSTER ? (int)cg::this_cluster().block_rank() : 0;
  const int i = blockIdx.y;
  const int blk = CLUSTER ? blockIdx.x / p.chunks : blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t d4 = p.d >> 2;
  const int64_t cg0 = (int64_t)rank * p.chunk4;
  const int64_t cg_end = min(d4, cg0 + p.chunk4);
  const int s_begin = blk * p.samples_per_block;
  const int s_end = min(p.m, s_begin + p.samples_per_block);

  float4 z[VPT], acc[VPT];
  bool valid[VPT];
#pragma unroll
  for (int j = 0; j < VPT; ++j) {
    const int64_t cgj = cg0 + threadIdx.x + (int64_t)j * T;
    valid[j] = cgj < cg_end;
    z[j] = valid[j] ? *reinterpret_cast<const float4 *>(p.Z + (int64_t)i * p.ld + cgj * 4)
                    : make_float4(0.f, 0.f, 0.f, 0.f);
    acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float *a_agent = p.A + (int64_t)i * p.m * p.d + cg0 * 4;
  const float *l_agent = p.labels + (int64_t)i * p.m;
  // every CTA of the cluster must be running before anybody writes into its shared memory
  if (CLUSTER) cg::this_cluster().sync();

  int buf = 0;
  for (int s = s_begin; s < s_end; s += NS) {
    float4 a[NS][VPT];
    float dot[NS];
#pragma unroll
    for (int jj = 0; jj < NS; ++jj) {
      const bool live = s + jj < s_end;
      const float *row = a_agent + (int64_t)(s + jj) * p.d;
#pragma unroll
      for (int j = 0; j < VPT; ++j) {
        const int64_t cgl = threadIdx.x + (int64_t)j * T;   // column group inside the chunk
        a[jj][j] = (live && valid[j]) ? __ldcs(reinterpret_cast<const float4 *>(row + cgl * 4))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
#pragma unroll
    for (int jj = 0; jj < NS; ++jj) {
      float t = 0.f;
#pragma unroll
      for (int j = 0; j < VPT; ++j) t += dot4(a[jj][j], z[j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
      dot[jj] = t;
    }
    if (lane == 0) red[buf][warp] = dots_pack(dot);
    __syncthreads();
    Dots tot = red[buf][0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) dots_add(tot, red[buf][w]);
    if (CLUSTER) {
      // tot is this CTA's share (its column chunk).  Thread t hands it to the CTA of rank t;
      // after the barrier every CTA adds the shares in rank order.  Two buffers: a CTA can only
      // write the next iteration's shares after everybody has read those of the previous one.
      cg::cluster_group cluster = cg::this_cluster();
      if ((int)threadIdx.x < p.chunks) *cluster.map_shared_rank(&share[buf][rank], threadIdx.x) = tot;
      cluster.sync();
      tot = share[buf][0];
      for (int r = 1; r < p.chunks; ++r) dots_add(tot, share[buf][r]);
    }
    float margin[NS];
    dots_unpack(tot, margin);
    buf ^= 1;  // the other buffer is free: everybody passed the barrier above after reading it
#pragma unroll
    for (int jj = 0; jj < NS; ++jj) {
      float coef = 0.f;
      if (s + jj < s_end) {
        coef = sample_coef<LOSS>(__ldg(l_agent + s + jj), margin[jj], p.inv_m);
      }
#pragma unroll
      for (int j = 0; j < VPT; ++j) {
        acc[j].x = fmaf(coef, a[jj][j].x, acc[j].x);
        acc[j].y = fmaf(coef, a[jj][j].y, acc[j].y);
        acc[j].z = fmaf(coef, a[jj][j].z, acc[j].z);
        acc[j].w = fmaf(coef, a[jj][j].w, acc[j].w);
      }
    }
  }
  float *out = p.partial + ((int64_t)i * p.P + blk) * p.d + cg0 * 4;
#pragma unroll
  for (int j = 0; j < VPT; ++j) {
    const int64_t cgl = threadIdx.x + (int64_t)j * T;
    if (valid[j]) *reinterpret_cast<float4 *>(out + cgl * 4) = acc[j];
  }
}

// G[i, c..c+3] = sum over the P partials, in block order (+ the caller's noise, if any).
__global__ void __launch_bounds__(256) logreg_reduce_kernel(const float *partial, const float *noise, float *G,
                                                            int32_t n, int32_t P, int64_t d, int64_t ld) {
  const int64_t d4 = d >> 2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * d4) return;
  const int64_t i = idx / d4, cg = idx - i * d4;
  const float *src = partial + i * P * d + cg * 4;
  float4 s = *reinterpret_cast<const float4 *>(src);
  for (int32_t b = 1; b < P; ++b) {
    const float4 v = *reinterpret_cast<const float4 *>(src + (int64_t)b * d);
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  if (noise) {
    const float4 e = *reinterpret_cast<const float4 *>(noise + i * ld + cg * 4);
    s.x += e.x; s.y += e.y; s.z += e.z; s.w += e.w;
  }
  *reinterpret_cast<float4 *>(G + i * ld + cg * 4) = s;
}

// ---- fallback: any d, any alignment ---------------------------------------------------------
template <int LOSS>
__global__ void __launch_bounds__(256) logreg_coef_kernel(const float *A, const float *labels, const float *Z,
                                                          float *coef, int32_t n, int32_t m, int64_t d, int64_t ld,
                                                          float inv_m) {
  const int64_t sample = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;  // one warp per sample
  const int lane = threadIdx.x & 31;
  if (sample >= (int64_t)n * m) return;
  const int64_t i = sample / m;
  const float *row = A + sample * d;
  const float *z = Z + i * ld;
  float t = 0.f;
  for (int64_t c = lane; c < d; c += 32) t = fmaf(row[c], z[c], t);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if (lane == 0) coef[sample] = sample_coef<LOSS>(labels[sample], t, inv_m);
}

__global__ void __launch_bounds__(256) logreg_accum_kernel(const float *A, const float *coef, const float *noise,
                                                           float *G, int32_t n, int32_t m, int64_t d, int64_t ld) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * d) return;
  const int64_t i = idx / d, c = idx - i * d;
  const float *col = A + i * m * d + c;
  const float *cf = coef + i * m;
  float g = 0.f;
  for (int32_t s = 0; s < m; ++s) g = fmaf(cf[s], col[(int64_t)s * d], g);
  if (noise) g += noise[i * ld + c];
  G[i * ld + c] = g;
}

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Kernels of the column-sharded form (defined further down); the two-pass fallback borrows them for rows
// too wide for a cluster.
__global__ void shard_dots_kernel(const float *A, const float *Z, float *dots, int32_t n, int32_t m, int64_t w,
                                  int64_t lda, int64_t ldz, int vec);
template <int LOSS>
__global__ void shard_coef_kernel(float *dots, const float *targets, int64_t count, float inv_m);
__global__ void shard_accum_vec_kernel(const float *A, const float *coef, const float *noise, float *G, int32_t m,
                                       int64_t w, int64_t lda, int64_t ldg);

size_t logreg_workspace_bytes(int32_t n, int32_t m, int64_t d) {
  const size_t partial = (size_t)n * (size_t)logreg_sample_blocks(n, m, d) * (size_t)d * sizeof(float);
  const size_t coef = (size_t)n * (size_t)m * sizeof(float);
  return ((partial + 255) / 256) * 256 + ((coef + 255) / 256) * 256;
}

// Enqueues the gradient kernels with `scratch` (>= logreg_workspace_bytes) as working memory.
// Nothing in the scratch has to start at zero: every partial sum and every coefficient that is read
// has been written earlier in the same call.
template <int LOSS>
static ceca_status_t enqueue_grad(const float *A, const float *targets, const float *Z, const float *noise, float *G,
                                  int32_t n, int32_t m, int64_t d, int64_t ld, void *scratch, cudaStream_t stream) {
  const float inv_m = (float)(1.0 / (double)m);
  const int32_t P = logreg_sample_blocks(n, m, d);
  float *partial = static_cast<float *>(scratch);
  const size_t partial_bytes = (((size_t)n * P * d * sizeof(float) + 255) / 256) * 256;
  float *coef = reinterpret_cast<float *>(static_cast<char *>(scratch) + partial_bytes);
  const int32_t chunks = logreg_chunks(d);
  const bool fast = (d % 4 == 0) && (ld % 4 == 0) && chunks <= kLrMaxCluster && aligned16(A) &&
                    aligned16(Z) && aligned16(G) && (!noise || aligned16(noise)) && n <= 65535;
  if (fast) {
    LogregArgs a;
    a.A = A; a.labels = targets; a.Z = Z; a.partial = partial;
    a.d = d; a.ld = ld; a.n = n; a.m = m; a.P = P;
    a.samples_per_block = (m + P - 1) / P;
    a.inv_m = inv_m;
    a.chunks = chunks;
    a.chunk4 = (d / 4 + chunks - 1) / chunks;
    const int threads = a.chunk4 > (int64_t)kLrThreads * kLrMaxVpt ? 2 * kLrThreads : kLrThreads;
    const int64_t groups = (a.chunk4 + threads - 1) / threads;   // float4 per thread and row
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)P * chunks, (unsigned)n);
    cfg.blockDim = dim3(threads);
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = chunks; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    if (chunks > 1) { cfg.attrs = &attr; cfg.numAttrs = 1; }
    cudaError_t e;
#define CECA_LR_LAUNCH(VPT_, CL_, T_) e = cudaLaunchKernelEx(&cfg, logreg_fused_kernel<VPT_, LOSS, CL_, T_>, a)
    if (threads > kLrThreads) {
      if (chunks > 1) CECA_LR_LAUNCH(4, true, 2 * kLrThreads); else CECA_LR_LAUNCH(4, false, 2 * kLrThreads);
    } else if (chunks > 1) {
      if (groups <= 1) CECA_LR_LAUNCH(1, true, kLrThreads);
      else if (groups <= 2) CECA_LR_LAUNCH(2, true, kLrThreads);
      else CECA_LR_LAUNCH(4, true, kLrThreads);
    } else {
      if (groups <= 1) CECA_LR_LAUNCH(1, false, kLrThreads);
      else if (groups <= 2) CECA_LR_LAUNCH(2, false, kLrThreads);
      else CECA_LR_LAUNCH(4, false, kLrThreads);
    }
#undef CECA_LR_LAUNCH
    if (e != cudaSuccess) return CECA_ERR_CUDA;
    const int64_t work = (int64_t)n * (d / 4);
    logreg_reduce_kernel<<<(unsigned)((work + 255) / 256), 256, 0, stream>>>(partial, noise, G, n, P, d, ld);
    return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
  }
  const int64_t blocks1 = ((int64_t)n * m * 32 + 255) / 256;
  const int64_t blocks2 = ((int64_t)n * d + 255) / 256;
  if (blocks1 > 0x7fffffffLL || blocks2 > 0x7fffffffLL) return CECA_ERR_UNSUPPORTED;
  if ((d % 4 == 0) && (ld % 4 == 0) && aligned16(A) && aligned16(Z) && aligned16(G) && (!noise || aligned16(noise)) &&
      n <= 65535) {
    // aligned rows wider than a cluster holds: A is read twice, both times with 128-bit streaming loads
    // (inner products, coefficients in place, then the A^T pass of 256 columns per CTA)
    const int64_t count = (int64_t)n * m;
    shard_dots_kernel<<<(unsigned)blocks1, 256, 0, stream>>>(A, Z, coef, n, m, d, d, ld, 1);
    if (cudaGetLastError() != cudaSuccess) return CECA_ERR_CUDA;
    shard_coef_kernel<LOSS><<<(unsigned)((count + 255) / 256), 256, 0, stream>>>(coef, targets, count, inv_m);
    if (cudaGetLastError() != cudaSuccess) return CECA_ERR_CUDA;
    const dim3 grid((unsigned)((d / 4 + 63) / 64), (unsigned)n);
    shard_accum_vec_kernel<<<grid, 256, 0, stream>>>(A, coef, noise, G, m, d, d, ld);
    return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
  }
  logreg_coef_kernel<LOSS><<<(unsigned)blocks1, 256, 0, stream>>>(A, targets, Z, coef, n, m, d, ld, inv_m);
  if (cudaGetLastError() != cudaSuccess) return CECA_ERR_CUDA;
  logreg_accum_kernel<<<(unsigned)blocks2, 256, 0, stream>>>(A, coef, noise, G, n, m, d, ld);
  return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

// Argument checks shared by the gradient entry points; picks z by the round of iteration k.
static ceca_status_t grad_args(const float *A, const float *targets, const float *X, const float *Y, int64_t k,
                               const float *G, int32_t n, int32_t m, int64_t d, int64_t ld, ceca_variant_t variant,
                               const float **Z) {
  if (!A || !targets || !X || !G || n < 1 || m < 1 || d < 1 || ld < d) return CECA_ERR_INVALID_ARG;
  Plan plan;
  ceca_status_t st = make_plan(n, variant, k, &plan);
  if (st != CECA_OK) return st;
  *Z = plan.rd.payload ? Y : X;
  return *Z ? CECA_OK : CECA_ERR_INVALID_ARG;
}

}  // namespace ceca

extern "C" ceca_status_t dsgd_logreg_grad(const float *A, const float *labels, const float *X, const float *Y,
                                          int64_t k, float *G, int32_t n, int32_t m, int64_t d, int64_t ld,
                                          ceca_variant_t variant, void *workspace, size_t workspace_bytes,
                                          void *stream) {
  using namespace ceca;
  const float *Z = nullptr;
  ceca_status_t st = grad_args(A, labels, X, Y, k, G, n, m, d, ld, variant, &Z);
  if (st != CECA_OK) return st;
  if (!workspace || workspace_bytes < logreg_workspace_bytes(n, m, d) || !aligned16(workspace))
    return CECA_ERR_WORKSPACE;
  return enqueue_grad<kLossLogistic>(A, labels, Z, nullptr, G, n, m, d, ld, workspace,
                                     static_cast<cudaStream_t>(stream));
}

extern "C" ceca_status_t dsgd_lsq_grad(const float *A, const float *B, const float *X, const float *Y,
                                       const float *noise, int64_t k, float *G, int32_t n, int32_t m, int64_t d,
                                       int64_t ld, ceca_variant_t variant, void *workspace, size_t workspace_bytes,
                                       void *stream) {
  using namespace ceca;
  const float *Z = nullptr;
  ceca_status_t st = grad_args(A, B, X, Y, k, G, n, m, d, ld, variant, &Z);
  if (st != CECA_OK) return st;
  if (!workspace || workspace_bytes < logreg_workspace_bytes(n, m, d) || !aligned16(workspace))
    return CECA_ERR_WORKSPACE;
  return enqueue_grad<kLossSquare>(A, B, Z, noise, G, n, m, d, ld, workspace, static_cast<cudaStream_t>(stream));
}

// ---- column-sharded form -----------------------------------------------------------------------
//
// When the parameter columns are split over several GPUs (the update itself mixes rows only, so a
// column block needs no exchange for it), a shard holds A[:, :, c0:c0+w] and z[:, c0:c0+w] and the
// gradient splits into (i) the partial inner products of the block, (ii) their sum over the shards
// (n x m floats: the one exchange per iteration, an all-reduce between GPUs) and (iii) the
// coefficient per sample and the block's share of A^T coef.  A is read once in (i) and once in (iii).
namespace ceca {

__global__ void __launch_bounds__(256) shard_dots_kernel(const float *A, const float *Z, float *dots, int32_t n,
                                                         int32_t m, int64_t w, int64_t lda, int64_t ldz, int vec) {
  const int64_t sample = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;  // one warp per sample
  const int lane = threadIdx.x & 31;
  if (sample >= (int64_t)n * m) return;
  const int64_t i = sample / m;
  const float *row = A + sample * lda;
  const float *z = Z + i * ldz;
  float t = 0.f;
  if (vec) {
    for (int64_t c = 4 * lane; c < w; c += 128)
      t += dot4(__ldcs(reinterpret_cast<const float4 *>(row + c)), *reinterpret_cast<const float4 *>(z + c));
  } else {
    for (int64_t c = lane; c < w; c += 32) t = fmaf(row[c], z[c], t);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  if (lane == 0) dots[sample] = t;
}

__global__ void __launch_bounds__(256) shard_sum_kernel(float *total, const float *part, int64_t count, int first) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < count) total[idx] = first ? part[idx] : total[idx] + part[idx];
}

template <int LOSS>
__global__ void __launch_bounds__(256) shard_coef_kernel(float *dots, const float *targets, int64_t count, float inv_m) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < count) dots[idx] = sample_coef<LOSS>(targets[idx], dots[idx], inv_m);
}

// G[i, :] = sum_s coef[i, s] * A[i, s, :] for 256 columns per CTA: a lane owns two float4 column groups 128
// columns apart (a warp reads two 512-byte pieces of a row), the eight warps take every eighth group of four
// samples and their sums are added in warp order through shared memory, so the result is the same from
// run to run.  Needs w, lda, ldg multiples of 4 and 16-byte aligned bases.
__global__ void __launch_bounds__(256) shard_accum_vec_kernel(const float *A, const float *coef, const float *noise,
                                                              float *G, int32_t m, int64_t w, int64_t lda, int64_t ldg) {
  constexpr int kRows = 4, kGroups = 2;
  __shared__ float4 part[8][kGroups][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t i = blockIdx.y;
  int64_t c[kGroups];
  bool live[kGroups];
  float4 acc[kGroups];
#pragma unroll
  for (int g = 0; g < kGroups; ++g) {
    c[g] = ((int64_t)blockIdx.x * kGroups * 32 + g * 32 + lane) * 4;
    live[g] = c[g] < w;
    acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float *rows = A + i * m * lda;
  const float *cf = coef + i * m;
  for (int32_t s0 = warp * kRows; s0 < m; s0 += 8 * kRows) {
    float4 a[kRows][kGroups];
    float k[kRows];
#pragma unroll
    for (int t = 0; t < kRows; ++t) {
      const bool ok = s0 + t < m;
      k[t] = ok ? __ldg(cf + s0 + t) : 0.f;
#pragma unroll
      for (int g = 0; g < kGroups; ++g)
        a[t][g] = (ok && live[g]) ? __ldcs(reinterpret_cast<const float4 *>(rows + (int64_t)(s0 + t) * lda + c[g]))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int t = 0; t < kRows; ++t)
#pragma unroll
      for (int g = 0; g < kGroups; ++g) {
        acc[g].x = fmaf(k[t], a[t][g].x, acc[g].x); acc[g].y = fmaf(k[t], a[t][g].y, acc[g].y);
        acc[g].z = fmaf(k[t], a[t][g].z, acc[g].z); acc[g].w = fmaf(k[t], a[t][g].w, acc[g].w);
      }
  }
#pragma unroll
  for (int g = 0; g < kGroups; ++g) part[warp][g][lane] = acc[g];
  __syncthreads();
  if (warp < kGroups && live[warp]) {   // warp g adds up column group g
    const int g = warp;
    float4 sum = part[0][g][lane];
#pragma unroll
    for (int v = 1; v < 8; ++v) { const float4 q = part[v][g][lane]; sum.x += q.x; sum.y += q.y; sum.z += q.z; sum.w += q.w; }
    if (noise) {
      const float4 e = *reinterpret_cast<const float4 *>(noise + i * ldg + c[g]);
      sum.x += e.x; sum.y += e.y; sum.z += e.z; sum.w += e.w;
    }
    *reinterpret_cast<float4 *>(G + i * ldg + c[g]) = sum;
  }
}

__global__ void __launch_bounds__(256) shard_accum_kernel(const float *A, const float *coef, const float *noise,
                                                          float *G, int32_t n, int32_t m, int64_t w, int64_t lda,
                                                          int64_t ldg) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * w) return;
  const int64_t i = idx / w, c = idx - i * w;
  const float *col = A + i * m * lda + c;
  const float *cf = coef + i * m;
  float g = 0.f;
  for (int32_t s = 0; s < m; ++s) g = fmaf(cf[s], col[(int64_t)s * lda], g);
  if (noise) g += noise[i * ldg + c];
  G[i * ldg + c] = g;
}

}  // namespace ceca

extern "C" ceca_status_t dsgd_grad_shard_dots(const float *A_shard, const float *Z_shard, float *dots, int32_t n,
                                              int32_t m, int64_t w, int64_t lda, int64_t ldz, void *stream) {
  using namespace ceca;
  if (!A_shard || !Z_shard || !dots || n < 1 || m < 1 || w < 1 || lda < w || ldz < w) return CECA_ERR_INVALID_ARG;
  const int64_t blocks = ((int64_t)n * m * 32 + 255) / 256;
  if (blocks > 0x7fffffffLL) return CECA_ERR_UNSUPPORTED;
  const int vec = (w % 4 == 0) && (lda % 4 == 0) && (ldz % 4 == 0) && aligned16(A_shard) && aligned16(Z_shard);
  shard_dots_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(A_shard, Z_shard, dots, n, m, w,
                                                                                      lda, ldz, vec);
  return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

extern "C" ceca_status_t dsgd_grad_shard_sum(float *total, const float *part, int64_t count, int32_t first,
                                             void *stream) {
  using namespace ceca;
  if (!total || !part || count < 1) return CECA_ERR_INVALID_ARG;
  const int64_t blocks = (count + 255) / 256;
  if (blocks > 0x7fffffffLL) return CECA_ERR_UNSUPPORTED;
  shard_sum_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(total, part, count, first != 0);
  return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

extern "C" ceca_status_t dsgd_grad_shard_apply(const float *A_shard, const float *targets, float *dots,
                                               const float *noise_shard, float *G_shard, int32_t n, int32_t m,
                                               int64_t w, int64_t lda, int64_t ldg, int32_t loss, void *stream) {
  using namespace ceca;
  if (!A_shard || !targets || !dots || !G_shard || n < 1 || m < 1 || w < 1 || lda < w || ldg < w)
    return CECA_ERR_INVALID_ARG;
  if (loss != kLossLogistic && loss != kLossSquare) return CECA_ERR_INVALID_ARG;
  const int64_t count = (int64_t)n * m;
  const int64_t blocks1 = (count + 255) / 256, blocks2 = ((int64_t)n * w + 255) / 256;
  if (blocks1 > 0x7fffffffLL || blocks2 > 0x7fffffffLL) return CECA_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const float inv_m = (float)(1.0 / (double)m);
  if (loss == kLossLogistic) shard_coef_kernel<kLossLogistic><<<(unsigned)blocks1, 256, 0, s>>>(dots, targets, count, inv_m);
  else shard_coef_kernel<kLossSquare><<<(unsigned)blocks1, 256, 0, s>>>(dots, targets, count, inv_m);
  if (cudaGetLastError() != cudaSuccess) return CECA_ERR_CUDA;
  const bool vec = (w % 4 == 0) && (lda % 4 == 0) && (ldg % 4 == 0) && aligned16(A_shard) && aligned16(G_shard) &&
                   (!noise_shard || aligned16(noise_shard)) && n <= 65535;
  if (vec) {
    const dim3 grid((unsigned)((w / 4 + 63) / 64), (unsigned)n);
    shard_accum_vec_kernel<<<grid, 256, 0, s>>>(A_shard, dots, noise_shard, G_shard, m, w, lda, ldg);
  } else {
    shard_accum_kernel<<<(unsigned)blocks2, 256, 0, s>>>(A_shard, dots, noise_shard, G_shard, n, m, w, lda, ldg);
  }
  return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

// ---- the same gradient for callers that cannot hand over a workspace ---------------------------
//
// Some callers have no way to get device memory at the moment they need the gradient: a plug-in
// whose host application owns the whole device heap, code that runs while a framework's caching
// allocator must not be re-entered, or a latency-critical loop in which cudaMalloc (which can
// synchronise the whole device) is off limits.  For them the partial sums and coefficients live
// in the fixed buffer below, which is part of the loaded module: every GPU on which this library
// is used holds these bytes from the first use until the process exits.
namespace ceca {

constexpr size_t kStaticScratchBytes = (size_t)32 << 20;  // 32 MiB: enough for n=63, m=2000, d=4096
static __device__ __align__(256) unsigned char g_logreg_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mutex;
static void *g_scratch_ptr[kMaxDevices];  // device address of g_logreg_scratch, per device ordinal

// In host code `g_logreg_scratch` is only a handle; the address a kernel can use has to be asked
// for, once per device, while that device is current.
static cudaError_t static_scratch_address(void **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void *ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_logreg_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace ceca

extern "C" size_t dsgd_logreg_grad_static_capacity(void) { return ceca::kStaticScratchBytes; }

extern "C" ceca_status_t dsgd_logreg_grad_static(const float *A, const float *labels, const float *X, const float *Y,
                                                 int64_t k, float *G, int32_t n, int32_t m, int64_t d, int64_t ld,
                                                 ceca_variant_t variant, void *stream) {
  using namespace ceca;
  const float *Z = nullptr;
  ceca_status_t st = grad_args(A, labels, X, Y, k, G, n, m, d, ld, variant, &Z);
  if (st != CECA_OK) return st;
  if (logreg_workspace_bytes(n, m, d) > kStaticScratchBytes) return CECA_ERR_STATIC_SCRATCH;  // nothing launched
  void *scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) return CECA_ERR_CUDA;
  return enqueue_grad<kLossLogistic>(A, labels, Z, nullptr, G, n, m, d, ld, scratch,
                                     static_cast<cudaStream_t>(stream));
}
