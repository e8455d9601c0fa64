// Fused CECA-2P consensus rounds (Sec. 3.1 "Main recursions", Algorithm 2) with register-resident
// blocks of agents: most of every round's exchange never leaves the register file, and what the
// kernel executes per value and round is close to the one fused multiply-add it has to do.
//
// Layout.  A CTA of P warps owns one 64-column tile of all n rows (TMA tensor load into shared
// memory).  A lane is two adjacent matrix columns; warp p keeps I and J of a contiguous block of
// agents (rows i0 .. i0+cnt-1) of those columns in registers, at static register positions.  The
// block size is a template argument CB = ceil(n / P): the first blocks hold CB agents, the others
// CB-1, so every loop over a block has a compile-time trip count and at most one predicated row.
//
// Why this cuts the exchange.  In round r of CECA-2P agent i receives from agent i - s with
// s = n_r + delta_r, and s roughly doubles every round (1, 2, 3, 6, 12, 24, 48 for n = 97).  While
// s is smaller than a block, row offset j >= s of a block receives from offset j - s of the same
// thread: a register-to-register update with compile-time indices (one instantiation of the round
// body per value of s, selected by a uniform switch).  Only the first s rows of a block need a
// value from the previous block, so only the last s rows of every block are published in shared
// memory.  Rounds with s >= block size exchange every row.  For n = 97 (blocks of 12-13 agents)
// that is (1+2+3+6+12)/13 + 2 = 3.9 full exchanges instead of 7.  All shared-memory accesses are
// 64-bit and conflict free (a warp touches 64 consecutive floats of one row), addressed as one
// base pointer plus compile-time offsets.
//
// Pipeline.  CTAs are persistent.  The first round reads the neighbours' payload straight from the
// landed tile (it holds exactly the not-yet-updated values), so it publishes nothing and needs no
// barrier; later rounds alternate between two exchange tiles, which makes one CTA barrier per round
// enough.  As soon as the landed tile is no longer needed (after the second round's barrier) the
// TMA load of the CTA's next tile is issued into it and overlaps the remaining rounds and the
// stores.  Results go straight from registers to global memory, 256 contiguous bytes per warp and row.
//
// Arithmetic.  Scaled variables I = alpha * Ih, J = beta * Jh:
//   I+ = a I + (1-a) z_src   becomes   Ih+ = Ih + cI * zh_src,  alpha+ = a * alpha,
//   J+ = b J + (1-b) z_src   becomes   Jh+ = Jh + cJ * zh_src,  beta+  = b * beta
// (b = 0, the first round of a cycle: Jh is cleared first, cJ = 1 and beta+ is the payload's scale),
// one packed fused multiply-add per pair of values and round; alpha, beta, cI, cJ are formed in fp64
// on the host and folded back into the values every 16 rounds and on output.  Within a thread the
// update runs from the highest row offset down, so that offset j - s still holds the value from
// before the round when offset j uses it.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>

#include "ceca.h"
#include "plan.h"
#include "tma.h"

namespace ceca {

constexpr int kBkTileCols = 64;
constexpr int kBkMaxRounds = 64;
constexpr int kBkRenormEvery = 16;
constexpr int kBkMaxCb = 16;
constexpr uint32_t kBkWaitPolls = 1u << 22;

struct BlockRound {
  float cI, cJ;        // Ih += cI * z_src, Jh += cJ * z_src
  float preI, preJ;    // when renorm: Ih *= preI, Jh *= preJ first
  int16_t hop;         // the shift s of this round
  uint8_t payload, jclear, renorm, partial;  // partial: s < smallest block, the in-register form applies
};

struct BlockArgs {
  float *Xo, *Yo;
  int64_t ld;
  int32_t d, n, rounds, has_y_in, has_y_out, tiles;
  int32_t nfull;       // blocks 0..nfull-1 hold CB agents, the others CB-1
  int32_t wait_polls;
  uint32_t tx_bytes;   // bytes the landing barrier is armed for
  float outI, outJ;
  int32_t *status;
  BlockRound rd[kBkMaxRounds];
};

__device__ __forceinline__ float2 axpy2(float2 c, float2 z, float2 acc) { return __ffma2_rn(c, z, acc); }

// One round with a compile-time shift S smaller than every block.  `buf` is this round's exchange
// tile, already offset to this thread's column pair; `full_block` says whether the block holds CB
// rows (else CB-1).
template <int CB, int S, bool PAYJ>
__device__ __forceinline__ void round_partial(float2 (&Ih)[CB], float2 (&Jh)[CB], float2 cI, float2 cJ, float *buf,
                                              bool publish, bool full_block, int i0, int src_row0) {
  float2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (publish) {
    // the last S rows of the block are what the next block's first S rows receive
    float2 *own = reinterpret_cast<float2 *>(buf + i0 * kBkTileCols);
    if (full_block) {
#pragma unroll
      for (int t = 0; t < S; ++t) own[(CB - S + t) * (kBkTileCols / 2)] = Z[CB - S + t];
    } else if constexpr (CB - 1 - S >= 0) {
#pragma unroll
      for (int t = 0; t < S; ++t) own[(CB - 1 - S + t) * (kBkTileCols / 2)] = Z[CB - 1 - S + t];
    }
    __syncthreads();
  }
  float2 R[S];
  const float2 *src = reinterpret_cast<const float2 *>(buf + src_row0 * kBkTileCols);  // S rows, no wrap inside
#pragma unroll
  for (int t = 0; t < S; ++t) R[t] = src[t * (kBkTileCols / 2)];
#pragma unroll
  for (int j = CB - 1; j >= S; --j) {  // descending: Z[j - S] is still the value from before this round
    const float2 z = Z[j - S];
    Ih[j] = axpy2(cI, z, Ih[j]);
    Jh[j] = axpy2(cJ, z, Jh[j]);
  }
#pragma unroll
  for (int t = 0; t < S; ++t) {
    Ih[t] = axpy2(cI, R[t], Ih[t]);
    Jh[t] = axpy2(cJ, R[t], Jh[t]);
  }
}

template <int CB, bool PAYJ>
__device__ __forceinline__ void dispatch_partial(int s, float2 (&Ih)[CB], float2 (&Jh)[CB], float2 cI, float2 cJ,
                                                 float *buf, bool publish, bool full_block, int i0, int src_row0) {
#define CECA_BK_CASE(S)                                                                             \
  case S:                                                                                           \
    if constexpr (S < CB) round_partial<CB, S, PAYJ>(Ih, Jh, cI, cJ, buf, publish, full_block, i0, src_row0); \
    break;
  switch (s) {
    CECA_BK_CASE(1) CECA_BK_CASE(2) CECA_BK_CASE(3) CECA_BK_CASE(4) CECA_BK_CASE(5) CECA_BK_CASE(6) CECA_BK_CASE(7)
    CECA_BK_CASE(8) CECA_BK_CASE(9) CECA_BK_CASE(10) CECA_BK_CASE(11) CECA_BK_CASE(12) CECA_BK_CASE(13)
    CECA_BK_CASE(14) CECA_BK_CASE(15)
    default: break;
  }
#undef CECA_BK_CASE
}

// One round in which every row receives through shared memory (s at least as large as a block).
template <int CB, bool PAYJ>
__device__ __forceinline__ void round_full(float2 (&Ih)[CB], float2 (&Jh)[CB], float2 cI, float2 cJ, float *buf,
                                           bool publish, bool full_block, int i0, int s, int n) {
  float2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (publish) {
    float2 *own = reinterpret_cast<float2 *>(buf + i0 * kBkTileCols);
#pragma unroll
    for (int j = 0; j < CB - 1; ++j) own[j * (kBkTileCols / 2)] = Z[j];
    if (full_block) own[(CB - 1) * (kBkTileCols / 2)] = Z[CB - 1];
    __syncthreads();
  }
  const int cnt = full_block ? CB : CB - 1;
  const int first = i0 - s;  // source row of offset 0, before the wrap-around
  float2 R[CB];
  if (first >= 0 || first + cnt <= 0) {  // the whole block on one side of the wrap-around
    const float2 *src = reinterpret_cast<const float2 *>(buf + (first >= 0 ? first : first + n) * kBkTileCols);
#pragma unroll
    for (int j = 0; j < CB - 1; ++j) R[j] = src[j * (kBkTileCols / 2)];
    R[CB - 1] = full_block ? src[(CB - 1) * (kBkTileCols / 2)] : make_float2(0.f, 0.f);
  } else {
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      int row = first + j;
      if (row < 0) row += n;
      R[j] = (j < cnt) ? *reinterpret_cast<const float2 *>(buf + row * kBkTileCols) : make_float2(0.f, 0.f);
    }
  }
#pragma unroll
  for (int j = 0; j < CB; ++j) {
    Ih[j] = axpy2(cI, R[j], Ih[j]);
    Jh[j] = axpy2(cJ, R[j], Jh[j]);
  }
}

// MINB = CTAs per SM the register allocation must allow.
template <int CB, int P, int MINB>
__global__ void __launch_bounds__(32 * P, MINB)
consensus_block_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                       const __grid_constant__ BlockArgs p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bar;
  const int n = p.n;
  const int lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  const int tile_floats = n * kBkTileCols;
  float *land_x = reinterpret_cast<float *>(smem_raw);   // [n][64] landed X tile
  float *xch_a = land_x + tile_floats;                   // [n][64] exchange tile of the odd rounds
  float *xch_b = xch_a + tile_floats;                    // [n][64] exchange tile of the even rounds
  float *land_y = xch_b + tile_floats;                   // [n][64] landed Y tile (only when Y is read)

  const bool full_block = part < p.nfull;
  const int cnt = full_block ? CB : CB - 1;
  const int i0 = full_block ? part * CB : p.nfull * CB + (part - p.nfull) * (CB - 1);
  const int colpair = 2 * lane;

  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue_load = [&](int32_t tile) {
    mbar_expect_tx(&bar, p.tx_bytes);
    tma_load_2d(land_x, &map_x, tile * kBkTileCols, 0, &bar);
    if (p.has_y_in) tma_load_2d(land_y, &map_y, tile * kBkTileCols, 0, &bar);
  };
  if (threadIdx.x == 0 && (int32_t)blockIdx.x < p.tiles) issue_load((int32_t)blockIdx.x);

  uint32_t phase = 0;
  for (int32_t tile = blockIdx.x; tile < p.tiles; tile += gridDim.x) {
    const bool landed = mbar_wait_bounded(&bar, phase, (uint32_t)p.wait_polls);
    // This barrier also separates the previous tile's last exchange reads from this tile's writes.
    if (!__syncthreads_and(landed)) {
      // The tile never arrived: flag it, give the transfer one more bounded chance to finish (so
      // that it cannot write into shared memory of a finished CTA) and give up without storing.
      if (threadIdx.x == 0) atomicExch(p.status, 1);
      mbar_wait_bounded(&bar, phase, (uint32_t)p.wait_polls);
      return;
    }
    phase ^= 1u;

    float2 Ih[CB], Jh[CB];
    {
      const float2 *own = reinterpret_cast<const float2 *>(land_x + i0 * kBkTileCols + colpair);
#pragma unroll
      for (int j = 0; j < CB - 1; ++j) Ih[j] = own[j * (kBkTileCols / 2)];
      Ih[CB - 1] = full_block ? own[(CB - 1) * (kBkTileCols / 2)] : make_float2(0.f, 0.f);
      if (p.has_y_in) {
        const float2 *owny = reinterpret_cast<const float2 *>(land_y + i0 * kBkTileCols + colpair);
#pragma unroll
        for (int j = 0; j < CB - 1; ++j) Jh[j] = owny[j * (kBkTileCols / 2)];
        Jh[CB - 1] = full_block ? owny[(CB - 1) * (kBkTileCols / 2)] : make_float2(0.f, 0.f);
      } else {
#pragma unroll
        for (int j = 0; j < CB; ++j) Jh[j] = make_float2(0.f, 0.f);
      }
    }
    const int32_t next_tile = tile + (int32_t)gridDim.x;
    const bool prefetch_in_loop = p.rounds > 2;

    for (int rnd = 0; rnd < p.rounds; ++rnd) {
      const BlockRound &rd = p.rd[rnd];
      if (rd.renorm) {
        const float sI = rd.preI, sJ = rd.preJ;
#pragma unroll
        for (int j = 0; j < CB; ++j) { Ih[j].x *= sI; Ih[j].y *= sI; Jh[j].x *= sJ; Jh[j].y *= sJ; }
      }
      if (rd.jclear) {
#pragma unroll
        for (int j = 0; j < CB; ++j) Jh[j] = make_float2(0.f, 0.f);
      }
      if (rnd == 2 && threadIdx.x == 0 && next_tile < p.tiles) {
        // every thread has passed the barrier of round 1, so all reads of the landed tile (own rows and
        // the first round's neighbours) are done: the next tile may land while this one is finished
        issue_load(next_tile);
      }
      const bool publish = rnd > 0;
      float *buf = (rnd == 0 ? (rd.payload ? land_y : land_x) : ((rnd & 1) ? xch_a : xch_b)) + colpair;
      const int s = rd.hop;
      const float2 cI = make_float2(rd.cI, rd.cI), cJ = make_float2(rd.cJ, rd.cJ);
      if (rd.partial) {
        const int src_row0 = (part == 0 ? n : i0) - s;
        if (rd.payload) dispatch_partial<CB, true>(s, Ih, Jh, cI, cJ, buf, publish, full_block, i0, src_row0);
        else            dispatch_partial<CB, false>(s, Ih, Jh, cI, cJ, buf, publish, full_block, i0, src_row0);
      } else {
        if (rd.payload) round_full<CB, true>(Ih, Jh, cI, cJ, buf, publish, full_block, i0, s, n);
        else            round_full<CB, false>(Ih, Jh, cI, cJ, buf, publish, full_block, i0, s, n);
      }
    }

    const int32_t col = tile * kBkTileCols + colpair;
    if (col < p.d) {
      const float oI = p.outI, oJ = p.outJ;
      const bool pair_ok = col + 1 < p.d;   // d odd: the last column has no partner
      float *dst = p.Xo + (int64_t)i0 * p.ld + col;
      float *dsty = p.Yo + (int64_t)i0 * p.ld + col;
#pragma unroll
      for (int j = 0; j < CB; ++j) {
        if (j < CB - 1 || full_block) {
          const float2 v = make_float2(oI * Ih[j].x, oI * Ih[j].y);
          if (pair_ok) __stcs(reinterpret_cast<float2 *>(dst + j * p.ld), v);
          else __stcs(dst + j * p.ld, v.x);
        }
      }
      if (p.has_y_out) {
#pragma unroll
        for (int j = 0; j < CB; ++j) {
          if (j < CB - 1 || full_block) {
            const float2 v = make_float2(oJ * Jh[j].x, oJ * Jh[j].y);
            if (pair_ok) __stcs(reinterpret_cast<float2 *>(dsty + j * p.ld), v);
            else __stcs(dsty + j * p.ld, v.x);
          }
        }
      }
    }
    if (!prefetch_in_loop && next_tile < p.tiles) {
      // fewer than three rounds: the landed tile was in use until the end
      __syncthreads();
      if (threadIdx.x == 0) issue_load(next_tile);
    }
  }
}

// ---- host side ----------------------------------------------------------------------------------

constexpr int kBkMaxRows = 256;
constexpr size_t kBkSmemLimit = 227 * 1024 - 1024;   // opt-in maximum per CTA minus the static part

// y_in: the first round reads Y, which takes a fourth shared-memory tile.
bool consensus_block_supports(int32_t n, ceca_variant_t variant, int32_t rounds, bool y_in) {
  return variant == CECA_2P && n >= 2 && n <= kBkMaxRows && rounds >= 1 && rounds <= kBkMaxRounds &&
         (size_t)(y_in ? 4 : 3) * n * kBkTileCols * sizeof(float) <= kBkSmemLimit;
}

template <int CB, int P, int MINB>
static cudaError_t launch_block(const CUtensorMap &mx, const CUtensorMap &my, BlockArgs &a, cudaStream_t stream) {
  const int n = a.n;
  a.nfull = n - P * (CB - 1);
  const int cmin = a.nfull == P ? CB : CB - 1;
  for (int t = 0; t < a.rounds; ++t) a.rd[t].partial = (a.rd[t].hop < cmin) ? 1 : 0;
  const size_t tile_bytes = (size_t)n * kBkTileCols * sizeof(float);
  const size_t smem = (a.has_y_in ? 4 : 3) * tile_bytes;
  constexpr size_t kMaxSmemWanted = (size_t)4 * CB * P * kBkTileCols * sizeof(float);
  constexpr size_t kMaxSmem = kMaxSmemWanted < kBkSmemLimit ? kMaxSmemWanted : kBkSmemLimit;
  if (smem > kMaxSmem) return cudaErrorInvalidConfiguration;
  static std::atomic<uint64_t> attr_done{0};
  cudaError_t e =
      set_max_shared_once(reinterpret_cast<const void *>(consensus_block_kernel<CB, P, MINB>), kMaxSmem, &attr_done);
  if (e != cudaSuccess) return e;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  // persistent CTAs: as many as fit on the device at once, not more than there are tiles
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, consensus_block_kernel<CB, P, MINB>, 32 * P, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const int64_t resident = (int64_t)sms * per_sm;
  const int grid = (int)(a.tiles < resident ? a.tiles : resident);
  consensus_block_kernel<CB, P, MINB><<<grid, 32 * P, smem, stream>>>(mx, my, a);
  return cudaGetLastError();
}

// Arguments are assumed validated by the caller (shapes, aliasing, 16-byte alignment of X / Y and
// ld % 4 == 0, d and ld within 32 bits, Y present when the first round reads it, status word).
// The caller has checked consensus_block_supports.
ceca_status_t consensus_block(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                              int64_t ld, int64_t k0, int32_t rounds, int32_t *status, int32_t wait_polls,
                              uint32_t tx_extra, cudaStream_t stream) {
  BlockArgs a;
  std::memset(&a, 0, sizeof(a));
  a.Xo = Xo; a.Yo = Yo; a.ld = ld; a.d = (int32_t)d; a.n = n; a.rounds = rounds;
  a.has_y_out = Yo ? 1 : 0;
  a.tiles = (int32_t)((d + kBkTileCols - 1) / kBkTileCols);
  a.status = status;
  a.wait_polls = wait_polls > 0 ? wait_polls : (int32_t)kBkWaitPolls;

  double alpha = 1.0, beta = 1.0;
  bool first_needs_y = false;
  for (int32_t t = 0; t < rounds; ++t) {
    Plan plan;
    ceca_status_t st = make_plan(n, CECA_2P, k0 + t, &plan);
    if (st != CECA_OK) return st;
    if (t == 0) first_needs_y = plan.reads_y;
    BlockRound &r = a.rd[t];
    if (t > 0 && t % kBkRenormEvery == 0) {  // fold the scales back so that the scaled values stay in range
      r.renorm = 1; r.preI = (float)alpha; r.preJ = (float)beta;
      alpha = 1.0; beta = 1.0;
    }
    const double wa = plan.rd.a, wb = plan.rd.b;
    const double zeta = plan.rd.payload ? beta : alpha;
    r.payload = (uint8_t)plan.rd.payload;
    r.hop = (int16_t)plan.walk.hop;
    r.cI = (float)((1.0 - wa) * zeta / (wa * alpha));
    if (plan.rd.b_num == 0) { r.jclear = 1; r.cJ = 1.f; }   // J+ = the received value: Jh = 0 + 1 * zh_src, beta+ = zeta
    else r.cJ = (float)((1.0 - wb) * zeta / (wb * beta));
    alpha = wa * alpha;
    beta = plan.rd.b_num == 0 ? zeta : wb * beta;
  }
  a.outI = (float)alpha; a.outJ = (float)beta;
  a.has_y_in = (Y != nullptr && first_needs_y) ? 1 : 0;
  a.tx_bytes = (uint32_t)n * kBkTileCols * sizeof(float) * (a.has_y_in ? 2u : 1u) + tx_extra;
  if (!consensus_block_supports(n, CECA_2P, rounds, a.has_y_in != 0)) return CECA_ERR_UNSUPPORTED;

  CUtensorMap mx, my;
  if (!tensor_map_2d(&mx, X, n, d, ld, kBkTileCols, n)) return CECA_ERR_CUDA;
  if (!tensor_map_2d(&my, a.has_y_in ? Y : X, n, d, ld, kBkTileCols, n)) return CECA_ERR_CUDA;

  cudaError_t e = cudaErrorInvalidValue;
  if (n <= 8 * kBkMaxCb) {
    switch ((n + 7) / 8) {   // 8 warps, blocks of ceil(n / 8) agents
      case 1: e = launch_block<1, 8, 4>(mx, my, a, stream); break;
      case 2: e = launch_block<2, 8, 4>(mx, my, a, stream); break;
      case 3: e = launch_block<3, 8, 4>(mx, my, a, stream); break;
      case 4: e = launch_block<4, 8, 4>(mx, my, a, stream); break;
      case 5: e = launch_block<5, 8, 4>(mx, my, a, stream); break;
      case 6: e = launch_block<6, 8, 4>(mx, my, a, stream); break;
      case 7: e = launch_block<7, 8, 3>(mx, my, a, stream); break;
      case 8: e = launch_block<8, 8, 3>(mx, my, a, stream); break;
      case 9: e = launch_block<9, 8, 3>(mx, my, a, stream); break;
      case 10: e = launch_block<10, 8, 3>(mx, my, a, stream); break;
      case 11: e = launch_block<11, 8, 2>(mx, my, a, stream); break;
      case 12: e = launch_block<12, 8, 2>(mx, my, a, stream); break;
      case 13: e = launch_block<13, 8, 2>(mx, my, a, stream); break;
      case 14: e = launch_block<14, 8, 2>(mx, my, a, stream); break;
      case 15: e = launch_block<15, 8, 2>(mx, my, a, stream); break;
      case 16: e = launch_block<16, 8, 2>(mx, my, a, stream); break;
    }
  } else {
    switch ((n + 15) / 16) {  // 16 warps, n = 129 .. 256
      case 9: e = launch_block<9, 16, 1>(mx, my, a, stream); break;
      case 10: e = launch_block<10, 16, 1>(mx, my, a, stream); break;
      case 11: e = launch_block<11, 16, 1>(mx, my, a, stream); break;
      case 12: e = launch_block<12, 16, 1>(mx, my, a, stream); break;
      case 13: e = launch_block<13, 16, 1>(mx, my, a, stream); break;
      case 14: e = launch_block<14, 16, 1>(mx, my, a, stream); break;
      case 15: e = launch_block<15, 16, 1>(mx, my, a, stream); break;
      case 16: e = launch_block<16, 16, 1>(mx, my, a, stream); break;
    }
  }
  if (e == cudaErrorInvalidConfiguration) return CECA_ERR_UNSUPPORTED;
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

}  // namespace ceca
