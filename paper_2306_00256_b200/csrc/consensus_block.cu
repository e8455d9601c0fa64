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
#include <type_traits>
#include <utility>

#include "ceca.h"
#include "plan.h"
#include "tma.h"

namespace ceca {

constexpr int kBkTileCols = 64;
constexpr int kBkMaxRounds = 64;
constexpr int kBkRenormEvery = 16;
constexpr int kBkMaxCb = 25;            // agents per block (100 state registers)
constexpr uint32_t kBkWaitPolls = 1u << 22;

constexpr int kBkPayloadJ = 1;  // the message is J (else I)
constexpr int kBkClearJ = 2;    // b = 0: J+ is the received value
constexpr int kBkRenorm = 4;    // fold the running scales back into the values first

struct BlockRound {
  float cI, cJ;        // Ih += cI * z_src, Jh += cJ * z_src
  float preI, preJ;    // with kBkRenorm: Ih *= preI, Jh *= preJ first
  int32_t hop;         // the shift s of this round
  int32_t mode;        // kBk* flags
  int32_t sel;         // which instantiation of the round body runs (see dispatch_round)
  int32_t pad;
};

struct BlockArgs {
  float *Xo, *Yo;
  int64_t ld;
  int32_t d, n, rounds, has_y_in, has_y_out, tiles;
  int32_t nfull;       // blocks 0..nfull-1 hold CB agents, the others CB-1
  int32_t single_xch;  // one exchange tile instead of two (saves shared memory, costs a second barrier per round)
  int32_t wait_polls;
  uint32_t tx_bytes;   // bytes the landing barrier is armed for
  float outI, outJ;
  int32_t *status;
  BlockRound rd[kBkMaxRounds];
};

// Two adjacent columns travel as one 64-bit value (low word = the even column), so that the state
// lives in aligned register pairs and the packed fp32 instructions take it without repacking.
typedef unsigned long long pk2;
__device__ __forceinline__ pk2 pk_make(float lo, float hi) {
  pk2 v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
  return v;
}
__device__ __forceinline__ float pk_lo(pk2 v) { return __uint_as_float((unsigned)(v & 0xffffffffull)); }
__device__ __forceinline__ pk2 axpy2(pk2 c, pk2 z, pk2 acc) {   // c * z + acc on both columns
  pk2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(c), "l"(z), "l"(acc));
  return d;
}
__device__ __forceinline__ pk2 mul2(pk2 c, pk2 v) {
  pk2 d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(c), "l"(v));
  return d;
}

// Compile-time loop: f(integral_constant<int, 0>), ..., f(integral_constant<int, N-1>).
template <int... Is, typename F>
__device__ __forceinline__ void static_for_impl(std::integer_sequence<int, Is...>, F &&f) {
  (f(std::integral_constant<int, Is>{}), ...);
}
template <int N, typename F>
__device__ __forceinline__ void static_for(F &&f) {
  static_for_impl(std::make_integer_sequence<int, N>{}, f);
}
#define CECA_IDX(I) decltype(I)::value

// Shared memory is addressed by 32-bit shared-window addresses with compile-time byte offsets, so
// that an access costs one instruction and no address arithmetic.
constexpr int kBkRowBytes = kBkTileCols * (int)sizeof(float);
template <int OFF>
__device__ __forceinline__ pk2 lds64(uint32_t addr) {
  pk2 v;
  asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(v) : "r"(addr), "n"(OFF) : "memory");
  return v;
}
template <int OFF>
__device__ __forceinline__ void sts64(uint32_t addr, pk2 v) {
  asm volatile("st.shared.b64 [%0+%1], %2;" ::"r"(addr), "n"(OFF), "l"(v) : "memory");
}

// What a thread knows about its place in the tile: shared addresses are those of the round's
// exchange tile, already offset to the thread's column pair.
struct BlockPos {
  uint32_t own;    // row i0 of the exchange tile
  uint32_t prev;   // in-register rounds: the row just after the S source rows (row i0; row n for block 0)
  uint32_t col;    // row 0
  int i0, cnt, n;
  bool full_block, publish;
};

// One round with a compile-time shift S smaller than every block.  Z (the payload) is Ih or Jh itself.
template <int CB, int S, bool PAYJ>
__device__ __forceinline__ void round_partial(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q) {
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (q.publish) {
    // the last S rows of the block are what the next block's first S rows receive
    if (q.full_block) {
      static_for<S>([&](auto T) { sts64<(CB - S + CECA_IDX(T)) * kBkRowBytes>(q.own, Z[CB - S + CECA_IDX(T)]); });
    } else if constexpr (CB - 1 - S >= 0) {
      static_for<S>([&](auto T) { sts64<(CB - 1 - S + CECA_IDX(T)) * kBkRowBytes>(q.own, Z[CB - 1 - S + CECA_IDX(T)]); });
    }
    __syncthreads();
  }
#pragma unroll
  for (int j = CB - 1; j >= S; --j) {  // descending: Z[j - S] is still the value from before this round
    const pk2 z = Z[j - S];
    Ih[j] = axpy2(cI, z, Ih[j]);
    Jh[j] = axpy2(cJ, z, Jh[j]);
  }
  // the first S rows receive from the S rows before the block (no wrap inside), eight loads in flight at a time
  constexpr int kChunk = 8;
  static_for<(S + kChunk - 1) / kChunk>([&](auto C) {
    constexpr int T0 = CECA_IDX(C) * kChunk;
    constexpr int TN = S - T0 < kChunk ? S - T0 : kChunk;
    pk2 R[TN];
    static_for<TN>([&](auto T) { R[CECA_IDX(T)] = lds64<(T0 + CECA_IDX(T) - S) * kBkRowBytes>(q.prev); });
    static_for<TN>([&](auto T) {
      Ih[T0 + CECA_IDX(T)] = axpy2(cI, R[CECA_IDX(T)], Ih[T0 + CECA_IDX(T)]);
      Jh[T0 + CECA_IDX(T)] = axpy2(cJ, R[CECA_IDX(T)], Jh[T0 + CECA_IDX(T)]);
    });
  });
}

// One round in which every row receives through shared memory (s at least as large as a block).
template <int CB, bool PAYJ>
__device__ __forceinline__ void round_full(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q, int s) {
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (q.publish) {
    static_for<CB - 1>([&](auto J) { sts64<CECA_IDX(J) * kBkRowBytes>(q.own, Z[CECA_IDX(J)]); });
    if (q.full_block) sts64<(CB - 1) * kBkRowBytes>(q.own, Z[CB - 1]);
    __syncthreads();
  }
  const int first = q.i0 - s;  // source row of offset 0, before the wrap-around
  if (first >= 0 || first + q.cnt <= 0) {  // the whole block on one side of the wrap-around
    const uint32_t src = q.col + (uint32_t)((first >= 0 ? first : first + q.n) * kBkRowBytes);
    constexpr int kChunk = 8;
    static_for<(CB + kChunk - 1) / kChunk>([&](auto C) {
      constexpr int J0 = CECA_IDX(C) * kChunk;
      constexpr int JN = CB - J0 < kChunk ? CB - J0 : kChunk;
      pk2 R[JN];
      static_for<JN>([&](auto J) {
        constexpr int row = J0 + CECA_IDX(J);
        if constexpr (row < CB - 1) R[CECA_IDX(J)] = lds64<row * kBkRowBytes>(src);
        else R[CECA_IDX(J)] = q.full_block ? lds64<row * kBkRowBytes>(src) : 0ull;
      });
      static_for<JN>([&](auto J) {
        Ih[J0 + CECA_IDX(J)] = axpy2(cI, R[CECA_IDX(J)], Ih[J0 + CECA_IDX(J)]);
        Jh[J0 + CECA_IDX(J)] = axpy2(cJ, R[CECA_IDX(J)], Jh[J0 + CECA_IDX(J)]);
      });
    });
  } else {
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      int row = first + j;
      if (row < 0) row += q.n;
      const pk2 r = (j < q.cnt) ? lds64<0>(q.col + (uint32_t)(row * kBkRowBytes)) : 0ull;
      Ih[j] = axpy2(cI, r, Ih[j]);
      Jh[j] = axpy2(cJ, r, Jh[j]);
    }
  }
}

// `sel` (formed on the host): 0 / 1 = every row through shared memory, payload I / J;
// 2 S + (0 / 1) = the in-register form with shift S, payload I / J.
template <int CB>
__device__ __forceinline__ void dispatch_round(int sel, int s, pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ,
                                               const BlockPos &q) {
#define CECA_BK_CASE(S)                                                              \
  case 2 * S:                                                                        \
    if constexpr (S < CB) round_partial<CB, S, false>(Ih, Jh, cI, cJ, q);            \
    break;                                                                           \
  case 2 * S + 1:                                                                    \
    if constexpr (S < CB) round_partial<CB, S, true>(Ih, Jh, cI, cJ, q);             \
    break;
  switch (sel) {
    case 0: round_full<CB, false>(Ih, Jh, cI, cJ, q, s); break;
    case 1: round_full<CB, true>(Ih, Jh, cI, cJ, q, s); break;
    CECA_BK_CASE(1) CECA_BK_CASE(2) CECA_BK_CASE(3) CECA_BK_CASE(4) CECA_BK_CASE(5) CECA_BK_CASE(6) CECA_BK_CASE(7)
    CECA_BK_CASE(8) CECA_BK_CASE(9) CECA_BK_CASE(10) CECA_BK_CASE(11) CECA_BK_CASE(12) CECA_BK_CASE(13)
    CECA_BK_CASE(14) CECA_BK_CASE(15) CECA_BK_CASE(16) CECA_BK_CASE(17) CECA_BK_CASE(18) CECA_BK_CASE(19)
    CECA_BK_CASE(20) CECA_BK_CASE(21) CECA_BK_CASE(22) CECA_BK_CASE(23) CECA_BK_CASE(24)
    default: break;
  }
#undef CECA_BK_CASE
}

// The number of warps (blocks of agents) per CTA is a launch parameter; MAXT only bounds it and
// thereby sets the register budget (65536 / MAXT registers per thread).
template <int CB, int MAXT>
__global__ void __launch_bounds__(MAXT, 1)
consensus_block_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                       const __grid_constant__ BlockArgs p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bar;
  const int n = p.n;
  const int lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  const uint32_t tile_bytes = (uint32_t)n * kBkRowBytes;
  // [n][64] tiles: landed X, exchange tile of the odd rounds, of the even rounds (the same tile when
  // there is only one), landed Y (when Y is read)
  const uint32_t sm_land_x = smem_u32(smem_raw);
  const uint32_t sm_xch_a = sm_land_x + tile_bytes, sm_xch_b = p.single_xch ? sm_xch_a : sm_xch_a + tile_bytes;
  const uint32_t y_tile = p.single_xch ? 2u : 3u;
  const uint32_t sm_land_y = sm_land_x + y_tile * tile_bytes;

  BlockPos q;
  q.n = n;
  q.full_block = part < p.nfull;
  q.cnt = q.full_block ? CB : CB - 1;
  q.i0 = q.full_block ? part * CB : p.nfull * CB + (part - p.nfull) * (CB - 1);
  const uint32_t col_off = 2u * lane * (uint32_t)sizeof(float);
  const uint32_t own_off = (uint32_t)q.i0 * kBkRowBytes + col_off;
  const uint32_t prev_off = (uint32_t)(part == 0 ? n : q.i0) * kBkRowBytes + col_off;

  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue_load = [&](int32_t tile) {
    mbar_expect_tx(&bar, p.tx_bytes);
    tma_load_2d(smem_raw, &map_x, tile * kBkTileCols, 0, &bar);
    if (p.has_y_in) tma_load_2d(smem_raw + (size_t)y_tile * tile_bytes, &map_y, tile * kBkTileCols, 0, &bar);
  };
  if (threadIdx.x == 0 && (int32_t)blockIdx.x < p.tiles) issue_load((int32_t)blockIdx.x);

  const bool prefetch_in_loop = p.rounds > 2;
  float *const dst_x = p.Xo + (int64_t)q.i0 * p.ld + 2 * lane;
  float *const dst_y = p.Yo + (int64_t)q.i0 * p.ld + 2 * lane;

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

    pk2 Ih[CB], Jh[CB];
    {
      const uint32_t own = sm_land_x + own_off;
      static_for<CB - 1>([&](auto J) { Ih[CECA_IDX(J)] = lds64<CECA_IDX(J) * kBkRowBytes>(own); });
      Ih[CB - 1] = q.full_block ? lds64<(CB - 1) * kBkRowBytes>(own) : 0ull;
      if (p.has_y_in) {
        const uint32_t owny = sm_land_y + own_off;
        static_for<CB - 1>([&](auto J) { Jh[CECA_IDX(J)] = lds64<CECA_IDX(J) * kBkRowBytes>(owny); });
        Jh[CB - 1] = q.full_block ? lds64<(CB - 1) * kBkRowBytes>(owny) : 0ull;
      } else {
#pragma unroll
        for (int j = 0; j < CB; ++j) Jh[j] = 0ull;
      }
    }
    const int32_t next_tile = tile + (int32_t)gridDim.x;

    for (int rnd = 0; rnd < p.rounds; ++rnd) {
      const BlockRound &rd = p.rd[rnd];
      const int mode = rd.mode;
      if (mode & (kBkRenorm | kBkClearJ)) {
        if (mode & kBkRenorm) {
          const pk2 sI = pk_make(rd.preI, rd.preI), sJ = pk_make(rd.preJ, rd.preJ);
#pragma unroll
          for (int j = 0; j < CB; ++j) { Ih[j] = mul2(sI, Ih[j]); Jh[j] = mul2(sJ, Jh[j]); }
        }
        if (mode & kBkClearJ) {
#pragma unroll
          for (int j = 0; j < CB; ++j) Jh[j] = 0ull;
        }
      }
      if (rnd == 2 && threadIdx.x == 0 && next_tile < p.tiles) {
        // every thread has passed the barrier of round 1, so all reads of the landed tile (own rows and
        // the first round's neighbours) are done: the next tile may land while this one is finished
        issue_load(next_tile);
      }
      // The first round finds every row's payload in the landed tile and publishes nothing.
      q.publish = rnd > 0;
      const uint32_t buf = rnd == 0 ? ((mode & kBkPayloadJ) ? sm_land_y : sm_land_x) : ((rnd & 1) ? sm_xch_a : sm_xch_b);
      q.own = buf + own_off;
      q.prev = buf + prev_off;
      q.col = buf + col_off;
      dispatch_round<CB>(rd.sel, rd.hop, Ih, Jh, pk_make(rd.cI, rd.cI), pk_make(rd.cJ, rd.cJ), q);
      // with a single exchange tile the next round's publish must wait for this round's reads
      if (p.single_xch && rnd >= 1 && rnd + 1 < p.rounds) __syncthreads();
    }

    const int32_t col = tile * kBkTileCols + 2 * lane;
    if (col + 1 < p.d) {
      const pk2 oI = pk_make(p.outI, p.outI), oJ = pk_make(p.outJ, p.outJ);
      float *dst = dst_x + col - 2 * lane;
#pragma unroll
      for (int j = 0; j < CB - 1; ++j) __stcs(reinterpret_cast<pk2 *>(dst + j * p.ld), mul2(oI, Ih[j]));
      if (q.full_block) __stcs(reinterpret_cast<pk2 *>(dst + (CB - 1) * p.ld), mul2(oI, Ih[CB - 1]));
      if (p.has_y_out) {
        float *dsty = dst_y + col - 2 * lane;
#pragma unroll
        for (int j = 0; j < CB - 1; ++j) __stcs(reinterpret_cast<pk2 *>(dsty + j * p.ld), mul2(oJ, Jh[j]));
        if (q.full_block) __stcs(reinterpret_cast<pk2 *>(dsty + (CB - 1) * p.ld), mul2(oJ, Jh[CB - 1]));
      }
    } else if (col < p.d) {   // d odd: the last column has no partner
#pragma unroll
      for (int j = 0; j < CB; ++j)
        if (j < q.cnt) {
          __stcs(p.Xo + (int64_t)(q.i0 + j) * p.ld + col, p.outI * pk_lo(Ih[j]));
          if (p.has_y_out) __stcs(p.Yo + (int64_t)(q.i0 + j) * p.ld + col, p.outJ * pk_lo(Jh[j]));
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

// y_in: the first round reads Y, which takes one more shared-memory tile (at least two are needed without it).
bool consensus_block_supports(int32_t n, ceca_variant_t variant, int32_t rounds, bool y_in) {
  return variant == CECA_2P && n >= 2 && n <= kBkMaxRows && rounds >= 1 && rounds <= kBkMaxRounds &&
         (size_t)(y_in ? 3 : 2) * n * kBkTileCols * sizeof(float) <= kBkSmemLimit;
}

constexpr int kBkMaxWarps = 12;   // 12 blocks of 22 agents cover n = 256

// Register budgets by block size (the state takes 4 * CB registers): a roomy one, and a lean one that
// still compiles without spilling to speak of.  65536 / kMaxThreads registers per thread.
template <int CB> struct BlockRegs {
  static constexpr int kRoomy = CB >= 15 ? 384 : CB >= 11 ? 640 : CB >= 7 ? 768 : 1024;
  static constexpr int kLean = CB >= 15 ? 512 : CB >= 11 ? 768 : 1024;
};

template <int CB, int MAXT>
static cudaError_t launch_block_regs(const CUtensorMap &mx, const CUtensorMap &my, const BlockArgs &a, int warps,
                                     size_t smem, int *per_sm_out, bool launch, cudaStream_t stream) {
  static std::atomic<uint64_t> attr_done{0};
  cudaError_t e = set_max_shared_once(reinterpret_cast<const void *>(consensus_block_kernel<CB, MAXT>), kBkSmemLimit,
                                      &attr_done);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, consensus_block_kernel<CB, MAXT>, 32 * warps, smem);
  if (e != cudaSuccess) return e;
  *per_sm_out = per_sm;
  if (!launch) return cudaSuccess;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  // persistent CTAs: as many as fit on the device at once, not more than there are tiles
  const int64_t resident = (int64_t)sms * per_sm;
  const int grid = (int)(a.tiles < resident ? a.tiles : resident);
  consensus_block_kernel<CB, MAXT><<<grid, 32 * warps, smem, stream>>>(mx, my, a);
  return cudaGetLastError();
}

template <int CB>
static cudaError_t launch_block(const CUtensorMap &mx, const CUtensorMap &my, BlockArgs &a, int warps,
                                cudaStream_t stream) {
  const int n = a.n;
  a.nfull = n - warps * (CB - 1);
  const int cmin = a.nfull == warps ? CB : CB - 1;
  for (int t = 0; t < a.rounds; ++t) {
    BlockRound &r = a.rd[t];
    const int pay = (r.mode & kBkPayloadJ) ? 1 : 0;
    r.sel = r.hop < cmin ? 2 * r.hop + pay : pay;   // in-register form while the shift is smaller than every block
  }
  const size_t tile_bytes = (size_t)n * kBkTileCols * sizeof(float);
  if (32 * warps > BlockRegs<CB>::kRoomy) return cudaErrorInvalidConfiguration;
  // Four candidates: two or one exchange tile, roomy or lean register budget.  The default is two tiles
  // and the roomy budget; an alternative is taken only when it lets more CTAs share an SM.
  constexpr int kRoomy = BlockRegs<CB>::kRoomy, kLean = BlockRegs<CB>::kLean;
  int best = 0, best_single = 0, best_lean = 0;
  for (int single = 0; single < 2; ++single) {
    const size_t smem = ((a.has_y_in ? 2 : 1) + (single ? 1 : 2)) * tile_bytes;
    if (smem > kBkSmemLimit) continue;
    int roomy = 0, lean = 0;
    cudaError_t e = launch_block_regs<CB, kRoomy>(mx, my, a, warps, smem, &roomy, false, stream);
    if (e != cudaSuccess) return e;
    if (kLean != kRoomy) {
      e = launch_block_regs<CB, kLean>(mx, my, a, warps, smem, &lean, false, stream);
      if (e != cudaSuccess) return e;
    }
    if (roomy > best) { best = roomy; best_single = single; best_lean = 0; }
    if (lean > best) { best = lean; best_single = single; best_lean = 1; }
  }
  if (best < 1) return cudaErrorInvalidConfiguration;
  a.single_xch = best_single;
  const size_t smem = ((a.has_y_in ? 2 : 1) + (best_single ? 1 : 2)) * tile_bytes;
  int per_sm = 0;
  if (best_lean) return launch_block_regs<CB, kLean>(mx, my, a, warps, smem, &per_sm, true, stream);
  return launch_block_regs<CB, kRoomy>(mx, my, a, warps, smem, &per_sm, true, stream);
}

// Blocks (= warps) per CTA for n agents.  As few, i.e. as large, as the register file allows (25
// agents take 100 state registers), because a round whose shift reaches the block size exchanges
// every row through shared memory and there are about log2(blocks) such rounds; and 1, 2 or a
// multiple of 4, so that the warps of a CTA, which move in lockstep from barrier to barrier, load
// the four schedulers of an SM evenly (5, 6, 7 or 9 warps measured 15-40 % slower than 4 or 8).
// `warps_override` > 0 forces a value (used to measure the alternatives).
static int block_warps(int n, int warps_override) {
  if (warps_override > 0) return warps_override;
  return n <= 25 ? 1 : n <= 50 ? 2 : n <= 100 ? 4 : n <= 200 ? 8 : 12;
}

// Arguments are assumed validated by the caller (shapes, aliasing, 16-byte alignment of X / Y and
// ld % 4 == 0, d and ld within 32 bits, Y present when the first round reads it, status word).
// The caller has checked consensus_block_supports.
ceca_status_t consensus_block(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                              int64_t ld, int64_t k0, int32_t rounds, int32_t *status, int32_t wait_polls,
                              uint32_t tx_extra, int warps_override, cudaStream_t stream) {
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
      r.mode |= kBkRenorm; r.preI = (float)alpha; r.preJ = (float)beta;
      alpha = 1.0; beta = 1.0;
    }
    const double wa = plan.rd.a, wb = plan.rd.b;
    const double zeta = plan.rd.payload ? beta : alpha;
    if (plan.rd.payload) r.mode |= kBkPayloadJ;
    r.hop = plan.walk.hop;
    r.cI = (float)((1.0 - wa) * zeta / (wa * alpha));
    if (plan.rd.b_num == 0) { r.mode |= kBkClearJ; r.cJ = 1.f; }   // J+ = the received value: Jh = 0 + 1 * zh_src, beta+ = zeta
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

  const int warps = block_warps(n, warps_override);
  if (warps < 1 || warps > kBkMaxWarps) return CECA_ERR_UNSUPPORTED;
  cudaError_t e = cudaErrorInvalidConfiguration;
  switch ((n + warps - 1) / warps) {   // agents per block
#define CECA_BK_LAUNCH(CB) case CB: e = launch_block<CB>(mx, my, a, warps, stream); break;
    CECA_BK_LAUNCH(1) CECA_BK_LAUNCH(2) CECA_BK_LAUNCH(3) CECA_BK_LAUNCH(4) CECA_BK_LAUNCH(5) CECA_BK_LAUNCH(6)
    CECA_BK_LAUNCH(7) CECA_BK_LAUNCH(8) CECA_BK_LAUNCH(9) CECA_BK_LAUNCH(10) CECA_BK_LAUNCH(11) CECA_BK_LAUNCH(12)
    CECA_BK_LAUNCH(13) CECA_BK_LAUNCH(14) CECA_BK_LAUNCH(15) CECA_BK_LAUNCH(16) CECA_BK_LAUNCH(17) CECA_BK_LAUNCH(18)
    CECA_BK_LAUNCH(19) CECA_BK_LAUNCH(20) CECA_BK_LAUNCH(21) CECA_BK_LAUNCH(22) CECA_BK_LAUNCH(23) CECA_BK_LAUNCH(24)
    CECA_BK_LAUNCH(25)
#undef CECA_BK_LAUNCH
    default: break;
  }
  if (e == cudaErrorInvalidConfiguration) return CECA_ERR_UNSUPPORTED;
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

}  // namespace ceca
