// CECA consensus rounds (Sec. 3.1 "Main recursions", Algorithm 2; Sec. 3.2 for the 1-port pairing).
//
// fused = 0: one pass of the step kernel (gamma = 0, no G) per round.
// fused = 1: one launch.  Three kernels; this file holds the dispatch and the one that exchanges every
//   row through shared memory (the register-block kernel and the tensor-memory kernel have files of
//   their own).  Each CTA brings an n x W column tile of X (and of Y when the first round needs it)
//   into shared memory with one TMA tensor load, moves it into registers (a thread keeps a few rows
//   of eight columns for the whole run), and runs all rounds on chip: per round every thread
//   publishes the payload (I or J) of its rows in a shared exchange buffer, the CTA synchronises,
//   and every thread picks up the value of the row it receives from.  Only 4 bytes per element per
//   round go through shared memory in each direction (128-bit accesses, packed two-wide fp32 FMAs;
//   eight columns per thread keep the index arithmetic per element small).  The finished tiles go
//   back with one TMA tensor store each.  HBM sees X once in and X (and Y) once out, instead of once
//   per round.  Several CTAs per SM overlap each other's load, compute and store phases.  Tiles are
//   32 columns wide for n <= 256 (one TMA box); for 256 < n <= 2048 they are 8 columns wide and made
//   of several boxes, so that all rows still fit in shared memory.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>

#include "ceca.h"
#include "plan.h"
#include "tma.h"

namespace ceca {

cudaError_t enqueue_step(const Plan &plan, const float *X, const float *Y, const float *G, float *Xo,
                         float *Yo, int32_t n, int64_t d, int64_t ld, float gamma,
                         cudaStream_t stream);
ceca_status_t check_matrix_args(const void *X, const void *X_out, int32_t n, int64_t d, int64_t ld);
bool consensus_block_supports(int32_t n, ceca_variant_t variant, int32_t rounds, bool y_in);
ceca_status_t consensus_block(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                              int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds, int32_t *status,
                              int32_t wait_polls, uint32_t tx_extra, int warps_override, cudaStream_t stream);
bool consensus_tmem_supports(int32_t n, int32_t rounds);
ceca_status_t consensus_tmem(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                             int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds, int32_t *status,
                             int32_t wait_polls, uint32_t tx_extra, cudaStream_t stream);

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
  int32_t wait_polls;       // poll budget of the bounded wait for the tile
  uint32_t tx_extra;        // added to the byte count the landing barrier is armed for (0 except in the self-test)
  int32_t *status;
  FusedRound rd[kMaxFusedRounds];
};

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
    mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t tile_bytes = (uint32_t)tile_rows * kTileCols * sizeof(float);  // boxes count in full
    mbar_expect_tx(&bar, (p.has_y_in ? 2 * tile_bytes : tile_bytes) + p.tx_extra);
    for (int b = 0; b < p.boxes; ++b) {  // rows past n are out of range for the tensor map: zero fill
      const int row0 = b * p.box_rows;
      tma_load_2d(tile_a + (size_t)row0 * kTileCols, &map_x_in, col0, row0, &bar);
      if (p.has_y_in) tma_load_2d(tile_b + (size_t)row0 * kTileCols, &map_y_in, col0, row0, &bar);
    }
  }
  const bool landed = mbar_wait_bounded(&bar, 0, (uint32_t)p.wait_polls);
  if (!__syncthreads_and(landed)) {  // one decision for the whole CTA
    // The transfer never arrived: flag it, give it one more bounded chance to land (so that
    // it cannot write into shared memory of a finished CTA), and give up without storing.
    if (threadIdx.x == 0) atomicExch(p.status, 1);
    mbar_wait_bounded(&bar, 0, (uint32_t)p.wait_polls);
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
template <int R, int W, int T>
static cudaError_t launch_fused(const CUtensorMap &mxi, const CUtensorMap &myi, const CUtensorMap &mxo,
                                const CUtensorMap &myo, const FusedArgs &args, int64_t d, cudaStream_t stream) {
  const size_t smem = 2 * (size_t)args.boxes * args.box_rows * W * sizeof(float);
  // the largest tile this instantiation is ever launched with: R rows for each of its row groups
  constexpr size_t kMaxSmem = 2 * (size_t)R * (T / (W / 8)) * W * sizeof(float);
  static std::atomic<uint64_t> attr_done{0};
  cudaError_t e = set_max_shared_once(reinterpret_cast<const void *>(consensus_fused_kernel<R, W, T>),
                                      kMaxSmem < smem ? smem : kMaxSmem, &attr_done);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (d + W - 1) / W;
  consensus_fused_kernel<R, W, T><<<(unsigned)tiles, T, smem, stream>>>(mxi, myi, mxo, myo, args);
  return cudaGetLastError();
}

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// `kind`: a ceca_fused_t other than CECA_UNFUSED.
// wait_polls <= 0: the default poll budget; tx_extra: see FusedArgs (self-test only).
static ceca_status_t consensus_fused(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                                     int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds, int kind,
                                     void *workspace, size_t workspace_bytes, int32_t wait_polls, uint32_t tx_extra,
                                     cudaStream_t stream) {
  if (n > kMaxFusedRows || rounds > kMaxFusedRounds || ld >= ((int64_t)1 << 32) || d > 0x7fffffffLL)
    return CECA_ERR_UNSUPPORTED;
  if (kind == CECA_FUSED_TMEM && !consensus_tmem_supports(n, rounds)) return CECA_ERR_UNSUPPORTED;

  if (!workspace || workspace_bytes < sizeof(int32_t) || !aligned16(workspace)) return CECA_ERR_WORKSPACE;
  FusedArgs args;
  std::memset(&args, 0, sizeof(args));
  args.n = n; args.rounds = rounds; args.one_port = (variant == CECA_1P);
  args.status = static_cast<int32_t *>(workspace);
  args.wait_polls = wait_polls > 0 ? wait_polls : (int32_t)kWaitPolls;
  args.tx_extra = tx_extra;
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

  const bool block_ok = consensus_block_supports(n, variant, rounds, args.has_y_in != 0);
  if (kind == CECA_FUSED_BLOCK && !block_ok) return CECA_ERR_UNSUPPORTED;
  if (kind == CECA_FUSED_BLOCK || (kind == CECA_FUSED_AUTO && block_ok))
    return consensus_block(X, args.has_y_in ? Y : nullptr, Xo, Yo, n, d, ld, variant, k0, rounds, args.status, wait_polls,
                           tx_extra, 0, stream);
  if (kind == CECA_FUSED_TMEM)
    return consensus_tmem(X, args.has_y_in ? Y : nullptr, Xo, Yo, n, d, ld, variant, k0, rounds, args.status,
                          wait_polls, tx_extra, stream);

  // tile geometry: all n rows, 32 columns wide while one TMA box (256 rows) holds them, else 8
  const int tile_cols = n <= kMaxBoxRows ? kWideTileCols : kNarrowTileCols;
  args.boxes = (n + kMaxBoxRows - 1) / kMaxBoxRows;
  args.box_rows = (n + args.boxes - 1) / args.boxes;
  if (tile_cols == kNarrowTileCols)  // every box must start on a 128-byte boundary of shared memory
    args.box_rows = (args.box_rows + 3) / 4 * 4;
  CUtensorMap mxi, myi, mxo, myo;
  if (!tensor_map_2d(&mxi, X, n, d, ld, tile_cols, args.box_rows) || !tensor_map_2d(&mxo, Xo, n, d, ld, tile_cols, args.box_rows))
    return CECA_ERR_CUDA;
  if (!tensor_map_2d(&myi, args.has_y_in ? Y : X, n, d, ld, tile_cols, args.box_rows)) return CECA_ERR_CUDA;
  if (!tensor_map_2d(&myo, Yo ? Yo : Xo, n, d, ld, tile_cols, args.box_rows)) return CECA_ERR_CUDA;

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

  if (fused < 0 || fused > CECA_FUSED_BLOCK) return CECA_ERR_INVALID_ARG;
  if (rounds == 0 || n == 1) {  // nothing to mix: the result is a copy of the input
    if (Y_out && !Y) return CECA_ERR_INVALID_ARG;
    cudaError_t e = cudaSuccess;
    if (X_out != X)
      e = cudaMemcpy2DAsync(X_out, ld * sizeof(float), X, ld * sizeof(float), d * sizeof(float), n,
                            cudaMemcpyDeviceToDevice, stream);
    if (e == cudaSuccess && Y_out && Y && Y_out != Y)
      e = cudaMemcpy2DAsync(Y_out, ld * sizeof(float), Y, ld * sizeof(float), d * sizeof(float), n,
                            cudaMemcpyDeviceToDevice, stream);
    return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
  }

  if (fused) {
    // the kernel takes at most kMaxFusedRounds rounds per launch: longer runs go in chunks, the
    // first from the inputs to the outputs, the others in place on the outputs
    if (rounds > kMaxFusedRounds && !Y_out) return CECA_ERR_UNSUPPORTED;  // Y has to live somewhere in between
    const float *x_in = X, *y_in = Y;
    for (int32_t done = 0; done < rounds; done += kMaxFusedRounds) {
      const int32_t chunk = rounds - done < kMaxFusedRounds ? rounds - done : kMaxFusedRounds;
      st = consensus_fused(x_in, y_in, X_out, Y_out, n, d, ld, variant, k0 + done, chunk, fused, workspace,
                           workspace_bytes, 0, 0, stream);
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

extern "C" ceca_status_t ceca_fused_wait_selftest(const float *X, float *X_out, int32_t n, int64_t d, int64_t ld,
                                                  int32_t fused, void *workspace, size_t workspace_bytes,
                                                  void *stream) {
  using namespace ceca;
  ceca_status_t st = check_matrix_args(X, X_out, n, d, ld);
  if (st != CECA_OK) return st;
  if (fused != CECA_FUSED_SMEM && fused != CECA_FUSED_TMEM && fused != CECA_FUSED_BLOCK) return CECA_ERR_INVALID_ARG;
  if ((const float *)X_out == X || n < 2) return CECA_ERR_UNSUPPORTED;
  // One round of CECA-2P from k0 = 0, with the landing barrier armed for 16 bytes more than the
  // tile delivers and a poll budget of a few thousand: the transfer itself completes normally,
  // only the wait cannot succeed.
  return consensus_fused(X, nullptr, X_out, nullptr, n, d, ld, CECA_2P, 0, 1, fused, workspace, workspace_bytes,
                         /*wait_polls=*/2048, /*tx_extra=*/16, static_cast<cudaStream_t>(stream));
}

extern "C" ceca_status_t ceca_read_status(const void *workspace, int32_t *status_out, void *stream) {
  if (!workspace || !status_out) return CECA_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(status_out, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return CECA_ERR_CUDA;
  return cudaStreamSynchronize(s) == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}
