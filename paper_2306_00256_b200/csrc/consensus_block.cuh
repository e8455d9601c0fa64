// Internal: the register-block fused consensus kernel and its launch templates, shared by the translation
// units that instantiate it (64-column 2-port tiles; narrower 2-port tiles; the 1-port form), so that they
// compile side by side.  The description of the kernel is at the top of consensus_block.cu.
#pragma once
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

constexpr int kBkMaxRounds = 64;
constexpr int kBkRenormEvery = 16;
constexpr int kBkMaxBoxRows = 256;      // a TMA box holds at most 256 rows; taller tiles land as several boxes
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
  int32_t blocks;      // blocks of agents
  int32_t nfull;       // balanced: blocks 0 .. nfull-1 hold CB agents, the others CB-1;
                       // uniform: blocks 0 .. nfull-1 (= blocks-1 or blocks) hold CB, the last one the rest
  int32_t boxes, box_rows;   // a tile lands as `boxes` TMA boxes of `box_rows` rows (boxes * box_rows >= n)
  uint32_t tile_bytes; // shared-memory footprint of one tile (a multiple of 128 that holds blocks * CB rows and all boxes)
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
// that an access costs one instruction and no address arithmetic.  RB = bytes per tile row.
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
  uint32_t next;   // 1-port rounds: the first row after the block (row 0 for the last block)
  uint32_t col;    // row 0
  int i0, cnt;     // cnt = real rows of the block (CB, fewer in the last block)
  bool full, publish;
};

// One round with a compile-time shift S smaller than a block.  Z (the payload) is Ih or Jh itself.
template <int CB, int RB, bool BAL, int CH, int S, bool PAYJ>
__device__ __forceinline__ void round_partial(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q) {
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (q.publish) {
    // the last S rows of a block are what the next block's first S rows receive
    if (q.full) {
      static_for<S>([&](auto T) { sts64<(CB - S + CECA_IDX(T)) * RB>(q.own, Z[CB - S + CECA_IDX(T)]); });
    } else if constexpr (BAL) {   // a block of CB - 1 rows
      if constexpr (CB - 1 - S >= 0)
        static_for<S>([&](auto T) { sts64<(CB - 1 - S + CECA_IDX(T)) * RB>(q.own, Z[CB - 1 - S + CECA_IDX(T)]); });
    } else {
      // the last block of the uniform cut publishes all its rows, wherever its real ones end
      // (block 0 finds them just below row n)
      static_for<CB>([&](auto J) { sts64<CECA_IDX(J) * RB>(q.own, Z[CECA_IDX(J)]); });
    }
    __syncthreads();
  }
#pragma unroll
  for (int j = CB - 1; j >= S; --j) {  // descending: Z[j - S] is still the value from before this round
    const pk2 z = Z[j - S];
    Ih[j] = axpy2(cI, z, Ih[j]);
    Jh[j] = axpy2(cJ, z, Jh[j]);
  }
  // the first S rows receive from the S rows before the block (no wrap inside), CH loads in flight at a time
  constexpr int kChunk = CH;
  static_for<(S + kChunk - 1) / kChunk>([&](auto C) {
    constexpr int T0 = CECA_IDX(C) * kChunk;
    constexpr int TN = S - T0 < kChunk ? S - T0 : kChunk;
    pk2 R[TN];
    static_for<TN>([&](auto T) { R[CECA_IDX(T)] = lds64<(T0 + CECA_IDX(T) - S) * RB>(q.prev); });
    static_for<TN>([&](auto T) {
      Ih[T0 + CECA_IDX(T)] = axpy2(cI, R[CECA_IDX(T)], Ih[T0 + CECA_IDX(T)]);
      Jh[T0 + CECA_IDX(T)] = axpy2(cJ, R[CECA_IDX(T)], Jh[T0 + CECA_IDX(T)]);
    });
  });
}

// One round in which every row receives through shared memory (s at least as large as a block).
// Uniform cut: phantom rows are published and updated like real ones; their addresses stay inside
// the tile (it holds blocks * CB rows), and what they receive is never used.
template <int CB, int RB, bool BAL, int CH, bool PAYJ>
__device__ __forceinline__ void round_full(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q, int s, int n) {
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (q.publish) {
    static_for<CB - 1>([&](auto J) { sts64<CECA_IDX(J) * RB>(q.own, Z[CECA_IDX(J)]); });
    if (!BAL || q.full) sts64<(CB - 1) * RB>(q.own, Z[CB - 1]);
    __syncthreads();
  }
  const int first = q.i0 - s;  // source row of offset 0, before the wrap-around
  if (first >= 0 || first + q.cnt <= 0) {  // the real rows of the block all on one side of the wrap-around
    const uint32_t src = q.col + (uint32_t)((first >= 0 ? first : first + n) * RB);
    constexpr int kChunk = CH;
    static_for<(CB + kChunk - 1) / kChunk>([&](auto C) {
      constexpr int J0 = CECA_IDX(C) * kChunk;
      constexpr int JN = CB - J0 < kChunk ? CB - J0 : kChunk;
      pk2 R[JN];
      static_for<JN>([&](auto J) {
        constexpr int row = J0 + CECA_IDX(J);
        if constexpr (!BAL || row < CB - 1) R[CECA_IDX(J)] = lds64<row * RB>(src);
        else R[CECA_IDX(J)] = q.full ? lds64<row * RB>(src) : 0ull;   // balanced: row CB-1 of a short block may lie outside the tile
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
      if (row < 0) row += n;
      const pk2 r = (j < q.cnt) ? lds64<0>(q.col + (uint32_t)(row * RB)) : 0ull;
      Ih[j] = axpy2(cI, r, Ih[j]);
      Jh[j] = axpy2(cJ, r, Jh[j]);
    }
  }
}

// `sel` (formed on the host): 0 / 1 = every row through shared memory, payload I / J;
// 2 S + (0 / 1) = the in-register form with shift S, payload I / J.
template <int CB, int RB, bool BAL, int CH>
__device__ __forceinline__ void dispatch_round(int sel, int s, int n, pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ,
                                               const BlockPos &q) {
#define CECA_BK_CASE(S)                                                              \
  case 2 * S:                                                                        \
    if constexpr (S < CB) round_partial<CB, RB, BAL, CH, S, false>(Ih, Jh, cI, cJ, q);        \
    break;                                                                           \
  case 2 * S + 1:                                                                    \
    if constexpr (S < CB) round_partial<CB, RB, BAL, CH, S, true>(Ih, Jh, cI, cJ, q);         \
    break;
  switch (sel) {
    case 0: round_full<CB, RB, BAL, CH, false>(Ih, Jh, cI, cJ, q, s, n); break;
    case 1: round_full<CB, RB, BAL, CH, true>(Ih, Jh, cI, cJ, q, s, n); break;
    CECA_BK_CASE(1) CECA_BK_CASE(2) CECA_BK_CASE(3) CECA_BK_CASE(4) CECA_BK_CASE(5) CECA_BK_CASE(6) CECA_BK_CASE(7)
    CECA_BK_CASE(8) CECA_BK_CASE(9) CECA_BK_CASE(10) CECA_BK_CASE(11) CECA_BK_CASE(12) CECA_BK_CASE(13)
    CECA_BK_CASE(14) CECA_BK_CASE(15) CECA_BK_CASE(16) CECA_BK_CASE(17) CECA_BK_CASE(18) CECA_BK_CASE(19)
    CECA_BK_CASE(20) CECA_BK_CASE(21) CECA_BK_CASE(22) CECA_BK_CASE(23) CECA_BK_CASE(24)
    default: break;
  }
#undef CECA_BK_CASE
}

// ---- CECA-1P (Sec. 3.2): pairwise exchange -------------------------------------------------------
// Round r pairs even row i with row i + o, o = 2 n_r + 1 (odd, modulo the even n): even rows receive
// from o rows further on, odd rows from o rows back, and the two rows of a pair swap their payloads.
// Blocks hold an even number of agents and start at even rows (sizes CB and CB - 2), so parity is a
// property of the register position: position 2p is an even row ("E_p"), 2p + 1 an odd one ("O_p").
// With h = n_r the pairing reads E_p <-> O_{p+h}: while h is smaller than a block, the pairs whose two
// rows lie in the same block swap in registers, the last h even rows of a block pair with the first h
// odd rows of the next one, and only those 2 h rows per block go through shared memory.

// One 1-port round with compile-time h = H smaller than every block (in pairs).
template <int CB, int RB, int CH, int H, bool PAYJ>
__device__ __forceinline__ void round_partial_1p(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q) {
  constexpr int C = CB / 2;   // pairs of positions in a full block; a short block has C - 1
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if constexpr (H > 0) {
    if (q.publish) {
      // the odd rows of the first H pairs (wanted by the block before) and the even rows of the last H pairs
      static_for<H>([&](auto T) { sts64<(2 * CECA_IDX(T) + 1) * RB>(q.own, Z[2 * CECA_IDX(T) + 1]); });
      if (q.full) {
        static_for<H>([&](auto T) { sts64<2 * (C - H + CECA_IDX(T)) * RB>(q.own, Z[2 * (C - H + CECA_IDX(T))]); });
      } else if constexpr (C - 1 - H >= 0) {
        static_for<H>([&](auto T) { sts64<2 * (C - 1 - H + CECA_IDX(T)) * RB>(q.own, Z[2 * (C - 1 - H + CECA_IDX(T))]); });
      }
      __syncthreads();
    }
  }
  // pairs inside the block: both rows read the other's value from before the round
  static_for<C - H>([&](auto P) {
    constexpr int e = 2 * CECA_IDX(P), o = 2 * (CECA_IDX(P) + H) + 1;
    if (q.full || CECA_IDX(P) < C - 1 - H) {   // in a short block the last pair of positions is not there
      const pk2 ze = Z[e], zo = Z[o];
      Ih[e] = axpy2(cI, zo, Ih[e]); Jh[e] = axpy2(cJ, zo, Jh[e]);
      Ih[o] = axpy2(cI, ze, Ih[o]); Jh[o] = axpy2(cJ, ze, Jh[o]);
    }
  });
  if constexpr (H > 0) {
    // the first H odd rows receive from the even rows 2 H - 1, 2 H - 3, ... rows before them (previous block)
    static_for<H>([&](auto T) {
      constexpr int o = 2 * CECA_IDX(T) + 1;
      const pk2 r = lds64<2 * (CECA_IDX(T) - H) * RB>(q.prev);
      Ih[o] = axpy2(cI, r, Ih[o]); Jh[o] = axpy2(cJ, r, Jh[o]);
    });
    // the last H even rows receive from the first H odd rows of the next block
    if (q.full) {
      static_for<H>([&](auto T) {
        constexpr int e = 2 * (C - H + CECA_IDX(T));
        const pk2 r = lds64<(2 * CECA_IDX(T) + 1) * RB>(q.next);
        Ih[e] = axpy2(cI, r, Ih[e]); Jh[e] = axpy2(cJ, r, Jh[e]);
      });
    } else if constexpr (C - 1 - H >= 0) {
      static_for<H>([&](auto T) {
        constexpr int e = 2 * (C - 1 - H + CECA_IDX(T));
        const pk2 r = lds64<(2 * CECA_IDX(T) + 1) * RB>(q.next);
        Ih[e] = axpy2(cI, r, Ih[e]); Jh[e] = axpy2(cJ, r, Jh[e]);
      });
    }
  }
}

// One 1-port round in which every row receives through shared memory (h at least as large as a block).
template <int CB, int RB, bool PAYJ>
__device__ __forceinline__ void round_full_1p(pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ, const BlockPos &q, int o, int n) {
  pk2(&Z)[CB] = PAYJ ? Jh : Ih;
  if (q.publish) {
    static_for<CB - 2>([&](auto J) { sts64<CECA_IDX(J) * RB>(q.own, Z[CECA_IDX(J)]); });
    if (q.full) { sts64<(CB - 2) * RB>(q.own, Z[CB - 2]); sts64<(CB - 1) * RB>(q.own, Z[CB - 1]); }
    __syncthreads();
  }
  // even rows read o rows further on, odd rows o rows back; each of the two streams is contiguous
  // unless the wrap-around at n falls inside it
  int fe = q.i0 + o, fo = q.i0 - o;
  const bool e_plain = fe + q.cnt <= n || fe >= n, o_plain = fo >= 0 || fo + q.cnt <= 0;
  if (fe >= n) fe -= n;
  if (fo + q.cnt <= 0) fo += n;
  if (e_plain && o_plain) {
    const uint32_t se = q.col + (uint32_t)(fe * RB), so = q.col + (uint32_t)(fo * RB);
    static_for<CB>([&](auto J) {
      constexpr int j = CECA_IDX(J);
      const pk2 r = (j < CB - 2 || q.full) ? lds64<j * RB>((j & 1) ? so : se) : 0ull;
      Ih[j] = axpy2(cI, r, Ih[j]); Jh[j] = axpy2(cJ, r, Jh[j]);
    });
  } else {
#pragma unroll
    for (int j = 0; j < CB; ++j) {
      int row = (j & 1) ? q.i0 + j - o : q.i0 + j + o;
      if (row < 0) row += n;
      if (row >= n) row -= n;
      const pk2 r = (j < q.cnt) ? lds64<0>(q.col + (uint32_t)(row * RB)) : 0ull;
      Ih[j] = axpy2(cI, r, Ih[j]); Jh[j] = axpy2(cJ, r, Jh[j]);
    }
  }
}

// `sel`: 0 / 1 = every row through shared memory, payload I / J; 2 (H + 1) + (0 / 1) = the in-register form.
template <int CB, int RB, int CH>
__device__ __forceinline__ void dispatch_round_1p(int sel, int o, int n, pk2 (&Ih)[CB], pk2 (&Jh)[CB], pk2 cI, pk2 cJ,
                                                  const BlockPos &q) {
#define CECA_BK_CASE(H)                                                                   \
  case 2 * (H + 1):                                                                       \
    if constexpr (H < CB / 2) round_partial_1p<CB, RB, CH, H, false>(Ih, Jh, cI, cJ, q);  \
    break;                                                                                \
  case 2 * (H + 1) + 1:                                                                   \
    if constexpr (H < CB / 2) round_partial_1p<CB, RB, CH, H, true>(Ih, Jh, cI, cJ, q);   \
    break;
  switch (sel) {
    case 0: round_full_1p<CB, RB, false>(Ih, Jh, cI, cJ, q, o, n); break;
    case 1: round_full_1p<CB, RB, true>(Ih, Jh, cI, cJ, q, o, n); break;
    CECA_BK_CASE(0) CECA_BK_CASE(1) CECA_BK_CASE(2) CECA_BK_CASE(3) CECA_BK_CASE(4) CECA_BK_CASE(5) CECA_BK_CASE(6)
    CECA_BK_CASE(7) CECA_BK_CASE(8) CECA_BK_CASE(9) CECA_BK_CASE(10) CECA_BK_CASE(11) CECA_BK_CASE(12)
    default: break;
  }
#undef CECA_BK_CASE
}

// CB agents per block, LPB threads (column pairs) per block.  The number of threads per CTA is a
// launch parameter; MAXT only bounds it and thereby sets the register budget (65536 / MAXT registers
// per thread).
// ONEP: the CECA-1P form (blocks of CB or CB - 2 agents, CB even; 64- and 32-column tiles).
template <int CB, int LPB, int MAXT, bool ONEP>
__global__ void __launch_bounds__(MAXT, 1)
consensus_block_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                       const __grid_constant__ BlockArgs p) {
  constexpr int kTileCols = 2 * LPB;
  constexpr int RB = kTileCols * (int)sizeof(float);
  constexpr bool kBalanced = LPB >= 16;
  // received rows in flight per thread: eight, or four where the state leaves fewer than 36 other registers
  constexpr int kInFlight = 65536 / MAXT - 4 * CB >= 36 ? 8 : 4;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bar;
  const int n = p.n;
  const int lane = threadIdx.x % LPB;       // column pair inside the tile
  const int part = LPB == 32 ? (int)(threadIdx.x / LPB) : min((int)(threadIdx.x / LPB), p.blocks - 1);
  // tiles of p.tile_bytes each: 0 = landed X, 1 = exchange tile of the odd rounds, 2 = of the even
  // rounds (tile 1 again when there is only one), then landed Y (when Y is read).  Tile addresses are
  // formed where they are used, from the kernel parameters, to keep registers for the state.
  const uint32_t sm_land_x = smem_u32(smem_raw);
  const uint32_t y_tile = p.single_xch ? 2u : 3u;

  BlockPos q;
  if (ONEP) {   // pairs of rows: the first p.nfull blocks hold CB / 2 of them, the others one less
    q.full = part < p.nfull;
    q.cnt = q.full ? CB : CB - 2;
    q.i0 = q.full ? part * CB : p.nfull * CB + (part - p.nfull) * (CB - 2);
  } else if (kBalanced) {
    q.full = part < p.nfull;
    q.cnt = q.full ? CB : CB - 1;
    q.i0 = q.full ? part * CB : p.nfull * CB + (part - p.nfull) * (CB - 1);
  } else {
    q.i0 = part * CB;
    q.cnt = min(CB, n - q.i0);
    q.full = q.cnt == CB;
  }
  const uint32_t col_off = 2u * lane * (uint32_t)sizeof(float);
  const uint32_t own_off = (uint32_t)q.i0 * RB + col_off;
  const uint32_t prev_off = (uint32_t)(part == 0 ? n : q.i0) * RB + col_off;
  // 1-port: the row after the block's last one (the last block is followed by row 0)
  const uint32_t next_off = (ONEP && part < p.blocks - 1) ? own_off + (uint32_t)q.cnt * RB : col_off;

  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    mbar_fence_init();
  }
  __syncthreads();

  auto issue_load = [&](int32_t tile) {
    mbar_expect_tx(&bar, p.tx_bytes);
    for (int b = 0; b < p.boxes; ++b) {   // rows past n are outside the tensor map: they read as zero
      const int row0 = b * p.box_rows;
      tma_load_2d(smem_raw + (size_t)row0 * RB, &map_x, tile * kTileCols, row0, &bar);
      if (p.has_y_in)
        tma_load_2d(smem_raw + (size_t)y_tile * p.tile_bytes + (size_t)row0 * RB, &map_y, tile * kTileCols, row0, &bar);
    }
  };
  if (threadIdx.x == 0 && (int32_t)blockIdx.x < p.tiles) issue_load((int32_t)blockIdx.x);

  const bool prefetch_in_loop = p.rounds > 2;

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
      // balanced cut: only row CB-1 may be missing; uniform cut: any number of rows of the last block
      const uint32_t own = sm_land_x + own_off, owny = own + y_tile * p.tile_bytes;
      if (!kBalanced && q.full) {
        static_for<CB>([&](auto J) { Ih[CECA_IDX(J)] = lds64<CECA_IDX(J) * RB>(own); });
      } else {
        static_for<CB>([&](auto J) {
          constexpr int j = CECA_IDX(J);
          if constexpr (kBalanced && j < CB - (ONEP ? 2 : 1)) Ih[j] = lds64<j * RB>(own);
          else Ih[j] = (q.full || j < q.cnt) ? lds64<j * RB>(own) : 0ull;
        });
      }
      if (!p.has_y_in) {
#pragma unroll
        for (int j = 0; j < CB; ++j) Jh[j] = 0ull;
      } else if (!kBalanced && q.full) {
        static_for<CB>([&](auto J) { Jh[CECA_IDX(J)] = lds64<CECA_IDX(J) * RB>(owny); });
      } else {
        static_for<CB>([&](auto J) {
          constexpr int j = CECA_IDX(J);
          if constexpr (kBalanced && j < CB - (ONEP ? 2 : 1)) Jh[j] = lds64<j * RB>(owny);
          else Jh[j] = (q.full || j < q.cnt) ? lds64<j * RB>(owny) : 0ull;
        });
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
      const uint32_t buf_tile = rnd == 0 ? ((mode & kBkPayloadJ) ? y_tile : 0u) : ((rnd & 1) || p.single_xch ? 1u : 2u);
      const uint32_t buf = sm_land_x + buf_tile * p.tile_bytes;
      q.own = buf + own_off;
      q.prev = buf + prev_off;
      q.col = buf + col_off;
      if constexpr (ONEP) {
        q.next = buf + next_off;
        dispatch_round_1p<CB, RB, kInFlight>(rd.sel, rd.hop, p.n, Ih, Jh, pk_make(rd.cI, rd.cI), pk_make(rd.cJ, rd.cJ), q);
      } else {
        dispatch_round<CB, RB, kBalanced, kInFlight>(rd.sel, rd.hop, p.n, Ih, Jh, pk_make(rd.cI, rd.cI), pk_make(rd.cJ, rd.cJ), q);
      }
      // with a single exchange tile the next round's publish must wait for this round's reads
      if (p.single_xch && rnd >= 1 && rnd + 1 < p.rounds) __syncthreads();
    }

    const int32_t col = tile * kTileCols + 2 * lane;
    // surplus threads (only where a block is narrower than a warp) shadow the last block and write nothing
    if (LPB < 32 && (int)(threadIdx.x / LPB) >= p.blocks) {
    } else if (col + 1 < p.d) {
      const pk2 oI = pk_make(p.outI, p.outI), oJ = pk_make(p.outJ, p.outJ);
      float *dst = p.Xo + (int64_t)q.i0 * p.ld + col;
      float *dsty = p.Yo + (int64_t)q.i0 * p.ld + col;
      if (!kBalanced && q.full) {
#pragma unroll
        for (int j = 0; j < CB; ++j) __stcs(reinterpret_cast<pk2 *>(dst + j * p.ld), mul2(oI, Ih[j]));
        if (p.has_y_out) {
#pragma unroll
          for (int j = 0; j < CB; ++j) __stcs(reinterpret_cast<pk2 *>(dsty + j * p.ld), mul2(oJ, Jh[j]));
        }
      } else {
        static_for<CB>([&](auto J) {
          constexpr int j = CECA_IDX(J);
          if ((kBalanced && j < CB - (ONEP ? 2 : 1)) || q.full || j < q.cnt) __stcs(reinterpret_cast<pk2 *>(dst + j * p.ld), mul2(oI, Ih[j]));
        });
        if (p.has_y_out) {
          static_for<CB>([&](auto J) {
            constexpr int j = CECA_IDX(J);
            if ((kBalanced && j < CB - (ONEP ? 2 : 1)) || q.full || j < q.cnt) __stcs(reinterpret_cast<pk2 *>(dsty + j * p.ld), mul2(oJ, Jh[j]));
          });
        }
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

// ---- launch templates ---------------------------------------------------------------------------

constexpr size_t kBkSmemLimit = 227 * 1024 - 1024;   // opt-in maximum per CTA minus the static part

// Register budgets by block size (the state takes 4 * CB registers): a roomy one, and a lean one that
// still compiles without spilling to speak of.  65536 / kMaxThreads registers per thread.
template <int CB> struct BlockRegs {
  static constexpr int kRoomy = CB >= 15 ? 384 : CB >= 11 ? 640 : CB >= 7 ? 768 : 1024;
  static constexpr int kLean = CB >= 26 ? 384 : CB >= 15 ? 512 : CB >= 11 ? 768 : 1024;
};

template <int CB, int LPB, int MAXT, bool ONEP>
static cudaError_t launch_block_regs(const CUtensorMap *maps, const BlockArgs &a, int threads,
                                     size_t smem, int *per_sm_out, bool launch, cudaStream_t stream) {
  static std::atomic<uint64_t> attr_done{0};
  cudaError_t e = set_max_shared_once(reinterpret_cast<const void *>(consensus_block_kernel<CB, LPB, MAXT, ONEP>),
                                      kBkSmemLimit, &attr_done);
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, consensus_block_kernel<CB, LPB, MAXT, ONEP>, threads, smem);
  if (e != cudaSuccess) return e;
  *per_sm_out = per_sm;
  if (!launch) return cudaSuccess;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  // persistent CTAs: as many as fit on the device at once, not more than there are tiles
  const int64_t resident = (int64_t)sms * per_sm;
  const int grid = (int)(a.tiles < resident ? a.tiles : resident);
  consensus_block_kernel<CB, LPB, MAXT, ONEP><<<grid, threads, smem, stream>>>(maps[0], maps[1], a);
  return cudaGetLastError();
}

// launch == false: only reports in *ctas_per_sm how many CTAs of the best launch shape share an SM.
template <int CB, int LPB, bool ONEP>
static cudaError_t launch_block(const CUtensorMap *maps, BlockArgs &a, int threads, int cmin, bool launch,
                                int *ctas_per_sm, cudaStream_t stream) {
  for (int t = 0; t < a.rounds; ++t) {
    BlockRound &r = a.rd[t];
    const int pay = (r.mode & kBkPayloadJ) ? 1 : 0;
    if (ONEP) {   // hop = 2 h + 1; cmin counts pairs of rows
      const int h = (r.hop - 1) / 2;
      r.sel = h < cmin ? 2 * (h + 1) + pay : pay;
    } else {
      r.sel = r.hop < cmin ? 2 * r.hop + pay : pay;   // in-register form while the shift is smaller than every block
    }
  }
  const size_t tile_bytes = a.tile_bytes;
  // Four candidates: two or one exchange tile, roomy or lean register budget.  The default is two tiles
  // and the roomy budget; an alternative is taken only when it lets more CTAs share an SM.
  constexpr int kRoomy = BlockRegs<CB>::kRoomy, kLean = BlockRegs<CB>::kLean;
  int best = 0, best_single = 0, best_lean = 0;
  for (int single = 0; single < 2; ++single) {
    const size_t smem = ((a.has_y_in ? 2 : 1) + (single ? 1 : 2)) * tile_bytes;
    if (smem > kBkSmemLimit) continue;
    int roomy = 0, lean = 0;
    if (threads <= kRoomy) {
      cudaError_t e = launch_block_regs<CB, LPB, kRoomy, ONEP>(maps, a, threads, smem, &roomy, false, stream);
      if (e != cudaSuccess) return e;
    }
    if (kLean != kRoomy && threads <= kLean) {
      cudaError_t e = launch_block_regs<CB, LPB, kLean, ONEP>(maps, a, threads, smem, &lean, false, stream);
      if (e != cudaSuccess) return e;
    }
    if (roomy > best) { best = roomy; best_single = single; best_lean = 0; }
    if (lean > best) { best = lean; best_single = single; best_lean = 1; }
  }
  *ctas_per_sm = best;
  if (best < 1) return cudaErrorInvalidConfiguration;
  if (!launch) return cudaSuccess;
  a.single_xch = best_single;
  const size_t smem = ((a.has_y_in ? 2 : 1) + (best_single ? 1 : 2)) * tile_bytes;
  int per_sm = 0;
  if (best_lean) return launch_block_regs<CB, LPB, kLean, ONEP>(maps, a, threads, smem, &per_sm, true, stream);
  return launch_block_regs<CB, LPB, kRoomy, ONEP>(maps, a, threads, smem, &per_sm, true, stream);
}

}  // namespace ceca
