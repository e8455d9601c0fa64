// CECA consensus rounds (Sec. 3.1 "Main recursions", Algorithm 2; Sec. 3.2 for the 1-port pairing).
//
// fused = 0: one pass of the step kernel (gamma = 0, no G) per round.
// fused = 1: one launch.  Each CTA brings an n x W column tile of X (and of Y when the first
//   round needs it) into shared memory with one TMA tensor load, moves it into registers (a
//   thread keeps a few rows of eight columns for the whole run), and runs all rounds on chip: per
//   round every thread publishes the payload (I or J) of its rows in a shared exchange buffer,
//   the CTA synchronises, and every thread picks up the value of the row it receives from.  Only
//   4 bytes per element per round go through shared memory in each direction (128-bit accesses,
//   packed two-wide fp32 FMAs; eight columns per thread keep the index arithmetic per element
//   small).  The finished tiles go back with one TMA tensor store each.  HBM sees X once in and
//   X (and Y) once out, instead of once per round.  Several CTAs per SM overlap each other's
//   load, compute and store phases.  Tiles are 32 columns wide for n <= 256 (one TMA box); for
//   256 < n <= 2048 they are 8 columns wide and made of several boxes, so that all rows still fit
//   in shared memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>

#include "ceca.h"
#include "plan.h"

namespace ceca {

cudaError_t enqueue_step(const Plan &plan, const float *X, const float *Y, const float *G, float *Xo,
                         float *Yo, int32_t n, int64_t d, int64_t ld, float gamma,
                         cudaStream_t stream);
ceca_status_t check_matrix_args(const void *X, const void *X_out, int32_t n, int64_t d, int64_t ld);

constexpr int kMaxFusedRounds = 64;
constexpr int kMaxBoxRows = 256;     // one TMA box holds at most 256 rows; taller tiles take several boxes
constexpr int kWideTileCols = 32;    // W for n <= 256: 128-byte row segments
constexpr int kNarrowTileCols = 8;   // W for 256 < n <= 2048: 32-byte row segments, so that all rows still fit
constexpr int kMaxFusedRows = 2048;
constexpr int kFusedThreads = 256;
constexpr uint32_t kWaitPolls = 1u << 22;  // bounded mbarrier wait (each poll sleeps ~100 ns)

struct FusedRound {
  int32_t hop;      // 2-port: shift s; 1-port: pairing offset o
  int32_t payload;  // 0: I is exchanged, 1: J
  float a, b, one_minus_a, one_minus_b;
};

struct FusedArgs {
  int32_t n, rounds, one_port, has_y_in, has_y_out;
  int32_t boxes, box_rows;  // the tile is `boxes` TMA boxes of `box_rows` rows (boxes * box_rows >= n)
  int32_t *status;
  FusedRound rd[kMaxFusedRounds];
};

// ---- PTX wrappers (mbarrier + TMA) ----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t phase) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(phase)
      : "memory");
  return ok != 0;
}
// Bounded wait: returns false when the barrier did not flip within the poll budget.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t phase, uint32_t polls) {
  for (uint32_t i = 0; i < polls; ++i) {
    if (mbar_try_wait(bar, phase)) return true;
    __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int32_t x, int32_t y,
                                            uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int32_t x, int32_t y, const void *src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(map), "r"(x), "r"(y), "r"(smem_u32(src))
               : "memory");
}

__device__ __forceinline__ float4 mix4(float w_own, float4 own, float w_recv, float4 recv) {
  // w_own * own + w_recv * recv on four lanes with two-wide packed fp32 instructions
  const float2 wo = make_float2(w_own, w_own), wr = make_float2(w_recv, w_recv);
  const float2 lo = __ffma2_rn(wo, make_float2(own.x, own.y), __fmul2_rn(wr, make_float2(recv.x, recv.y)));
  const float2 hi = __ffma2_rn(wo, make_float2(own.z, own.w), __fmul2_rn(wr, make_float2(recv.z, recv.w)));
  return make_float4(lo.x, lo.y, hi.x, hi.y);
}

// R = rows per thread, W = tile width in columns (both compile time).
//
// Thread layout: a thread owns eight columns (two float4) of each of its rows.  With COLG = W / 8
// column groups per row and Q = T / COLG row groups (T threads per CTA): cg = tid % COLG, q = tid / COLG, rows
// q, q + Q, ..., so n <= R * Q.  The two float4 of a row sit at column groups cg and cg + COLG; a
// thread touches them in that order or swapped, depending on a bit of q chosen such that the eight
// threads sharing a 128-bit shared-memory transaction cover all 32 banks:
//   W = 32 (rows 128 bytes apart): two adjacent row groups share a transaction -> swap on q & 1;
//   W = 8  (rows  32 bytes apart): eight adjacent rows share it              -> swap on (q >> 2) & 1.
template <int R, int W, int T>
__global__ void __launch_bounds__(T)
consensus_fused_kernel(const __grid_constant__ CUtensorMap map_x_in, const __grid_constant__ CUtensorMap map_y_in,
                       const __grid_constant__ CUtensorMap map_x_out,
                       const __grid_constant__ CUtensorMap map_y_out, const __grid_constant__ FusedArgs p) {
  constexpr int kTileCols = W;
  constexpr int kColGroups = W / 8;
  constexpr int kRowGroups = T / kColGroups;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = p.n;
  float *tile_a = reinterpret_cast<float *>(smem_raw);            // [n][W]  X tile, then exchange buffer
  const int tile_rows = p.boxes * p.box_rows;                     // >= n; the surplus rows are never used
  float *tile_b = tile_a + (size_t)tile_rows * kTileCols;         // [n][W]  Y tile, then exchange buffer
  __shared__ __align__(8) uint64_t bar;

  const int cg = threadIdx.x % kColGroups;
  const int q = threadIdx.x / kColGroups;
  const int swap = (W == 32) ? (q & 1) : ((q >> 2) & 1);
  const int c0 = 4 * (cg + kColGroups * swap);        // columns of the float4 touched first
  const int c1 = 4 * (cg + kColGroups * (swap ^ 1));  // ... and second
  const int32_t col0 = (int32_t)blockIdx.x * kTileCols;  // a multiple of 8 floats: 16-byte aligned

  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t tile_bytes = (uint32_t)tile_rows * kTileCols * sizeof(float);  // boxes count in full
    mbar_expect_tx(&bar, p.has_y_in ? 2 * tile_bytes : tile_bytes);
    for (int b = 0; b < p.boxes; ++b) {  // rows past n are out of range for the tensor map: zero fill
      const int row0 = b * p.box_rows;
      tma_load_2d(tile_a + (size_t)row0 * kTileCols, &map_x_in, col0, row0, &bar);
      if (p.has_y_in) tma_load_2d(tile_b + (size_t)row0 * kTileCols, &map_y_in, col0, row0, &bar);
    }
  }
  const bool landed = mbar_wait_bounded(&bar, 0, kWaitPolls);
  if (!__syncthreads_and(landed)) {  // one decision for the whole CTA
    // The transfer never arrived: flag it, give it one more bounded chance to land (so that
    // it cannot write into shared memory of a finished CTA), and give up without storing.
    if (threadIdx.x == 0) atomicExch(p.status, 1);
    mbar_wait_bounded(&bar, 0, kWaitPolls);
    return;
  }

  float4 I0[R], I1[R], J0[R], J1[R];
#pragma unroll
  for (int t = 0; t < R; ++t) {
    const int i = q + t * kRowGroups;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    I0[t] = I1[t] = J0[t] = J1[t] = zero;
    if (i < n) {
      I0[t] = *reinterpret_cast<const float4 *>(tile_a + i * kTileCols + c0);
      I1[t] = *reinterpret_cast<const float4 *>(tile_a + i * kTileCols + c1);
      if (p.has_y_in) {
        J0[t] = *reinterpret_cast<const float4 *>(tile_b + i * kTileCols + c0);
        J1[t] = *reinterpret_cast<const float4 *>(tile_b + i * kTileCols + c1);
      }
    }
  }
  // The landed tiles double as the first round's exchange buffer: if that round sends I it reads
  // tile_a as it is, if it sends J it reads tile_b (present whenever J carries data).  Later rounds
  // alternate between the two tiles, starting with the one the first round does not read.
  const int first_buf = (p.rounds > 0 && p.rd[0].payload && p.has_y_in) ? 1 : 0;
  const bool first_free = p.rounds > 0 && (!p.rd[0].payload || p.has_y_in);

  for (int rnd = 0; rnd < p.rounds; ++rnd) {
    const FusedRound rd = p.rd[rnd];
    float *buf = ((rnd + first_buf) & 1) ? tile_b : tile_a;
    if (rnd == 0 && first_free) {
      // nothing to publish: every thread has passed the landing barrier, the tile is complete
    } else if (rd.payload) {
#pragma unroll
      for (int t = 0; t < R; ++t) {
        const int i = q + t * kRowGroups;
        if (i < n) {
          *reinterpret_cast<float4 *>(buf + i * kTileCols + c0) = J0[t];
          *reinterpret_cast<float4 *>(buf + i * kTileCols + c1) = J1[t];
        }
      }
    } else {
#pragma unroll
      for (int t = 0; t < R; ++t) {
        const int i = q + t * kRowGroups;
        if (i < n) {
          *reinterpret_cast<float4 *>(buf + i * kTileCols + c0) = I0[t];
          *reinterpret_cast<float4 *>(buf + i * kTileCols + c1) = I1[t];
        }
      }
    }
    __syncthreads();  // payloads visible; in round 0 also: everybody has taken its own rows out
#pragma unroll
    for (int t = 0; t < R; ++t) {
      const int i = q + t * kRowGroups;
      if (i < n) {
        int src;
        if (p.one_port && !(i & 1)) { src = i + rd.hop; if (src >= n) src -= n; }
        else                        { src = i - rd.hop; if (src < 0) src += n; }
        const float4 r0 = *reinterpret_cast<const float4 *>(buf + src * kTileCols + c0);
        const float4 r1 = *reinterpret_cast<const float4 *>(buf + src * kTileCols + c1);
        I0[t] = mix4(rd.a, I0[t], rd.one_minus_a, r0);
        I1[t] = mix4(rd.a, I1[t], rd.one_minus_a, r1);
        J0[t] = mix4(rd.b, J0[t], rd.one_minus_b, r0);
        J1[t] = mix4(rd.b, J1[t], rd.one_minus_b, r1);
      }
    }
    // no second barrier: the next round writes the other buffer, and a thread can only start
    // the round after that once everybody has passed the next round's barrier.
  }
  __syncthreads();  // the last round's reads are done: the tiles can take the results

#pragma unroll
  for (int t = 0; t < R; ++t) {
    const int i = q + t * kRowGroups;
    if (i < n) {
      *reinterpret_cast<float4 *>(tile_a + i * kTileCols + c0) = I0[t];
      *reinterpret_cast<float4 *>(tile_a + i * kTileCols + c1) = I1[t];
      if (p.has_y_out) {
        *reinterpret_cast<float4 *>(tile_b + i * kTileCols + c0) = J0[t];
        *reinterpret_cast<float4 *>(tile_b + i * kTileCols + c1) = J1[t];
      }
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to TMA
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int b = 0; b < p.boxes; ++b) {  // the tensor map clips rows >= n and columns >= d
      const int row0 = b * p.box_rows;
      tma_store_2d(&map_x_out, col0, row0, tile_a + (size_t)row0 * kTileCols);
      if (p.has_y_out) tma_store_2d(&map_y_out, col0, row0, tile_b + (size_t)row0 * kTileCols);
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // smem must outlive the reads
  }
}

// ---- host side ------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(sym);
  }();
  return fn;
}

// An n x d fp32 matrix with row pitch ld, boxed as box_rows rows x tile_cols columns.
static bool make_map(CUtensorMap *map, const float *base, int32_t n, int64_t d, int64_t ld, int tile_cols,
                     int box_rows) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)n};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)tile_cols, (cuuint32_t)box_rows};
  const cuuint32_t elem[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, elem,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int R, int W, int T>
static cudaError_t launch_fused(const CUtensorMap &mxi, const CUtensorMap &myi, const CUtensorMap &mxo,
                                const CUtensorMap &myo, const FusedArgs &args, int64_t d, cudaStream_t stream) {
  const size_t smem = 2 * (size_t)args.boxes * args.box_rows * W * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(consensus_fused_kernel<R, W, T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(consensus_fused_kernel<R, W, T>, cudaFuncAttributePreferredSharedMemoryCarveout,
                           cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (d + W - 1) / W;
  consensus_fused_kernel<R, W, T><<<(unsigned)tiles, T, smem, stream>>>(mxi, myi, mxo, myo, args);
  return cudaGetLastError();
}

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static ceca_status_t consensus_fused(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                                     int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds,
                                     void *workspace, size_t workspace_bytes, cudaStream_t stream) {
  if (n > kMaxFusedRows || rounds > kMaxFusedRounds || ld >= ((int64_t)1 << 32) || d > 0x7fffffffLL)
    return CECA_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < sizeof(int32_t) || !aligned16(workspace)) return CECA_ERR_WORKSPACE;
  FusedArgs args;
  std::memset(&args, 0, sizeof(args));
  args.n = n; args.rounds = rounds; args.one_port = (variant == CECA_1P);
  args.status = static_cast<int32_t *>(workspace);
  bool first_needs_y = false;
  for (int32_t t = 0; t < rounds; ++t) {
    Plan plan;
    ceca_status_t st = make_plan(n, variant, k0 + t, &plan);
    if (st != CECA_OK) return st;
    if (t == 0) first_needs_y = plan.reads_y;
    FusedRound &r = args.rd[t];
    r.hop = plan.walk.hop;  // 2-port: the shift; 1-port: the pairing offset
    r.payload = plan.rd.payload;
    r.a = plan.a; r.b = plan.b; r.one_minus_a = plan.one_minus_a; r.one_minus_b = plan.one_minus_b;
  }
  if (first_needs_y && !Y) return CECA_ERR_INVALID_ARG;
  args.has_y_in = (Y != nullptr && first_needs_y) ? 1 : 0;
  args.has_y_out = Yo ? 1 : 0;
  if ((ld % 4) != 0 || !aligned16(X) || !aligned16(Xo) || (args.has_y_in && !aligned16(Y)) ||
      (Yo && !aligned16(Yo)))
    return CECA_ERR_ALIGNMENT;

  // tile geometry: all n rows, 32 columns wide while one TMA box (256 rows) holds them, else 8
  const int tile_cols = n <= kMaxBoxRows ? kWideTileCols : kNarrowTileCols;
  args.boxes = (n + kMaxBoxRows - 1) / kMaxBoxRows;
  args.box_rows = (n + args.boxes - 1) / args.boxes;
  if (tile_cols == kNarrowTileCols)  // every box must start on a 128-byte boundary of shared memory
    args.box_rows = (args.box_rows + 3) / 4 * 4;
  CUtensorMap mxi, myi, mxo, myo;
  if (!make_map(&mxi, X, n, d, ld, tile_cols, args.box_rows) || !make_map(&mxo, Xo, n, d, ld, tile_cols, args.box_rows))
    return CECA_ERR_CUDA;
  if (!make_map(&myi, args.has_y_in ? Y : X, n, d, ld, tile_cols, args.box_rows)) return CECA_ERR_CUDA;
  if (!make_map(&myo, Yo ? Yo : Xo, n, d, ld, tile_cols, args.box_rows)) return CECA_ERR_CUDA;

  cudaError_t e;
  if (tile_cols == kWideTileCols) {
    const int rows_per_thread = (n + 63) / 64;  // 64 row groups; n <= 256 -> at most 4
    if (rows_per_thread <= 1)      e = launch_fused<1, kWideTileCols, kFusedThreads>(mxi, myi, mxo, myo, args, d, stream);
    else if (rows_per_thread <= 2) e = launch_fused<2, kWideTileCols, kFusedThreads>(mxi, myi, mxo, myo, args, d, stream);
    else if (rows_per_thread <= 3) e = launch_fused<3, kWideTileCols, kFusedThreads>(mxi, myi, mxo, myo, args, d, stream);
    else                           e = launch_fused<4, kWideTileCols, kFusedThreads>(mxi, myi, mxo, myo, args, d, stream);
  } else {
    constexpr int kNarrowThreads = 512;  // one row group per thread: more warps per SM for the exchange loop
    const int rows_per_thread = (n + kNarrowThreads - 1) / kNarrowThreads;  // n <= 2048 -> at most 4
    if (rows_per_thread <= 1)      e = launch_fused<1, kNarrowTileCols, kNarrowThreads>(mxi, myi, mxo, myo, args, d, stream);
    else if (rows_per_thread <= 2) e = launch_fused<2, kNarrowTileCols, kNarrowThreads>(mxi, myi, mxo, myo, args, d, stream);
    else if (rows_per_thread <= 3) e = launch_fused<3, kNarrowTileCols, kNarrowThreads>(mxi, myi, mxo, myo, args, d, stream);
    else                           e = launch_fused<4, kNarrowTileCols, kNarrowThreads>(mxi, myi, mxo, myo, args, d, stream);
  }
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

}  // namespace ceca

extern "C" ceca_status_t ceca_consensus_rounds(const float *X, const float *Y, float *X_out, float *Y_out,
                                               int32_t n, int64_t d, int64_t ld, ceca_variant_t variant,
                                               int64_t k0, int32_t rounds, int32_t fused, void *workspace,
                                               size_t workspace_bytes, void *stream_) {
  using namespace ceca;
  ceca_status_t st = check_matrix_args(X, X_out, n, d, ld);
  if (st != CECA_OK) return st;
  if (rounds < 0 || k0 < 0) return CECA_ERR_INVALID_ARG;
  if (X_out == Y_out || (const float *)X_out == Y || (Y_out && (const float *)Y_out == X))
    return CECA_ERR_UNSUPPORTED;
  Plan first;
  st = make_plan(n, variant, k0, &first);  // also validates the variant / parity of n
  if (st != CECA_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);

  if (rounds == 0 || n == 1) {  // nothing to mix: the result is a copy of the input
    cudaError_t e = cudaSuccess;
    if (X_out != X)
      e = cudaMemcpy2DAsync(X_out, ld * sizeof(float), X, ld * sizeof(float), d * sizeof(float), n,
                            cudaMemcpyDeviceToDevice, stream);
    if (e == cudaSuccess && Y_out && Y && Y_out != Y)
      e = cudaMemcpy2DAsync(Y_out, ld * sizeof(float), Y, ld * sizeof(float), d * sizeof(float), n,
                            cudaMemcpyDeviceToDevice, stream);
    if (Y_out && !Y) return CECA_ERR_INVALID_ARG;
    return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
  }

  if (fused) {
    // the kernel takes at most kMaxFusedRounds rounds per launch: longer runs go in chunks, the
    // first from the inputs to the outputs, the others in place on the outputs
    if (rounds > kMaxFusedRounds && !Y_out) return CECA_ERR_UNSUPPORTED;  // Y has to live somewhere in between
    const float *x_in = X, *y_in = Y;
    for (int32_t done = 0; done < rounds; done += kMaxFusedRounds) {
      const int32_t chunk = rounds - done < kMaxFusedRounds ? rounds - done : kMaxFusedRounds;
      st = consensus_fused(x_in, y_in, X_out, Y_out, n, d, ld, variant, k0 + done, chunk, workspace,
                           workspace_bytes, stream);
      if (st != CECA_OK) return st;
      x_in = X_out; y_in = Y_out;
    }
    return CECA_OK;
  }

  if (!Y_out && (n & (n - 1)) == 0) {
    // n a power of two and Y not wanted back: every round sends I, so J never matters; run the
    // x-only form of the step kernel (8 bytes per element and round, no workspace)
    const float *x_src = X;
    for (int32_t t = 0; t < rounds; ++t) {
      Plan plan;
      st = make_plan(n, variant, k0 + t, &plan);
      if (st != CECA_OK) return st;
      if (enqueue_step(plan, x_src, nullptr, nullptr, X_out, nullptr, n, d, ld, 0.f, stream) != cudaSuccess)
        return CECA_ERR_CUDA;
      x_src = X_out;
    }
    return CECA_OK;
  }
  if (!Y && first.reads_y) return CECA_ERR_INVALID_ARG;
  float *y_work = Y_out;
  if (!y_work) {  // the caller does not want Y back: keep it in the workspace
    if (!workspace || workspace_bytes < (size_t)n * (size_t)ld * sizeof(float)) return CECA_ERR_WORKSPACE;
    y_work = static_cast<float *>(workspace);
    if ((const float *)y_work == X || (const float *)y_work == Y || y_work == X_out) return CECA_ERR_UNSUPPORTED;
  }
  const float *x_in = X, *y_in = Y;
  for (int32_t t = 0; t < rounds; ++t) {
    Plan plan;
    st = make_plan(n, variant, k0 + t, &plan);
    if (st != CECA_OK) return st;
    cudaError_t e = enqueue_step(plan, x_in, y_in, nullptr, X_out, y_work, n, d, ld, 0.f, stream);
    if (e != cudaSuccess) return CECA_ERR_CUDA;
    x_in = X_out; y_in = y_work;  // later rounds run in place on the outputs
  }
  return CECA_OK;
}

extern "C" ceca_status_t ceca_read_status(const void *workspace, int32_t *status_out, void *stream) {
  if (!workspace || !status_out) return CECA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(status_out, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return CECA_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}
