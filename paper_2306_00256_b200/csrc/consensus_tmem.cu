// Fused CECA consensus rounds (Sec. 3.1 "Main recursions", Algorithm 2; Sec. 3.2 for the 1-port
// pairing) for n <= 128 agents, with the per-round exchange going through Blackwell tensor memory
// instead of shared memory.
//
// Why tensor memory.  With all rounds on chip the only per-round traffic is the exchange: every
// row publishes its payload (I or J) and picks up the payload of the row it receives from.  Through
// shared memory that is one store and one load per element and round, and at n = 97 these fill
// the shared-memory pipe for longer than HBM needs to stream the matrix.  Tensor memory is a
// second on-chip store with its own datapath to the register file (tcgen05.st / tcgen05.ld; no
// tensor-core instruction is involved).  Its access rule fits the problem: a warp reaches only the
// 32 lanes of its own quadrant, but the four warps w, w+4, w+8, w+12 of a CTA share a quadrant,
// and a lane's columns are addressed dynamically.  So a tensor-memory lane is made one matrix
// column, a tensor-memory column one agent, and the four warps of a quadrant split the agents into
// four contiguous blocks: a thread keeps I and J of up to 32 consecutive agents of one matrix
// column in registers, publishes its block with a few tcgen05.st, and reads the block it receives
// from -- the same agents shifted by the round's hop, i.e. the same lane at a column offset -- with
// a few tcgen05.ld.  The wrap-around of the shift is handled by storing the first block of agents
// a second time behind the last one.
//
// Structure.  A CTA is four independent groups (one per quadrant = per SM sub-partition) of four
// warps; each group walks over 32-column tiles of the matrix: TMA tensor load of the n x 32 tile
// into shared memory (the next tile is prefetched while the rounds of the current one run), own
// rows to registers, all rounds with named-barrier synchronisation inside the group only, results
// straight from registers to global memory (a warp writes one full 128-byte line per row).  HBM
// sees X once in and X (and Y) once out.
//
// Arithmetic.  The rounds run on scaled variables I = alpha * Ih, J = beta * Jh:
//   I+ = a I + (1-a) r   becomes   Ih+ = Ih + cI * rh,  alpha+ = a * alpha,
//   J+ = b J + (1-b) r   becomes   Jh+ = Jh + cJ * rh,  beta+  = b * beta   (b = 0: Jh+ = rh),
// one fused multiply-add per value and round, with the scalars alpha, beta, cI, cJ formed in fp64 on
// the host; the scales are folded back every 16 rounds and at the end.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstring>
#include <type_traits>

#include "ceca.h"
#include "plan.h"
#include "tma.h"

namespace ceca {

constexpr int kTmThreads = 512;          // 16 warps: 4 quadrant groups x 4 row blocks
constexpr int kTmParts = 4;
constexpr int kTmTileCols = 32;          // matrix columns per group tile = lanes of a quadrant
constexpr int kTmMaxCnt = 32;            // agents per thread
constexpr int kTmMaxRows = kTmParts * kTmMaxCnt;
constexpr int kTmMaxRounds = 64;
constexpr int kTmRenormEvery = 16;
constexpr uint32_t kTmWaitPolls = 1u << 22;

struct TmemRound {
  float cI, cJ;          // Ih += cI * rh;  Jh += cJ * rh (or Jh = rh when jcopy)
  float preI, preJ;      // when renorm: Ih *= preI, Jh *= preJ before the round
  int16_t rdcol[kTmParts];  // per row block: first tensor-memory column (within a buffer) of its source range
  uint8_t payload, jcopy, renorm, pad;
};

struct TmemArgs {
  float *Xo, *Yo;
  int64_t ld;
  int32_t d, n, rounds, has_y_in, has_y_out, tiles;
  int32_t rstride;                // rows between consecutive agents of a block: 1 (2-port), 2 (1-port)
  int32_t buf_cols, alloc_cols;   // tensor-memory columns per exchange buffer / allocated
  int32_t wait_polls;             // poll budget of the bounded TMA wait
  uint32_t tx_bytes;              // bytes the TMA loads of one tile deliver
  int16_t stcol[kTmParts], cnt[kTmParts], row0[kTmParts], dupoff[kTmParts];
  float outI, outJ;               // X_out = outI * Ih, Y_out = outJ * Jh
  int32_t *status;
  TmemRound rd[kTmMaxRounds];
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------
template <int N> using IC = std::integral_constant<int, N>;

#define TM_F1(r, b) "f"(r[b])
#define TM_F2(r, b) TM_F1(r, b), TM_F1(r, b + 1)
#define TM_F4(r, b) TM_F2(r, b), TM_F2(r, b + 2)
#define TM_F8(r, b) TM_F4(r, b), TM_F4(r, b + 4)
#define TM_F16(r, b) TM_F8(r, b), TM_F8(r, b + 8)
#define TM_O1(r, b) "=f"(r[b])
#define TM_O2(r, b) TM_O1(r, b), TM_O1(r, b + 1)
#define TM_O4(r, b) TM_O2(r, b), TM_O2(r, b + 2)
#define TM_O8(r, b) TM_O4(r, b), TM_O4(r, b + 4)
#define TM_O16(r, b) TM_O8(r, b), TM_O8(r, b + 8)
#define TM_P1(r, b) "+f"(r[b])
#define TM_P2(r, b) TM_P1(r, b), TM_P1(r, b + 1)
#define TM_P4(r, b) TM_P2(r, b), TM_P2(r, b + 2)
#define TM_P8(r, b) TM_P4(r, b), TM_P4(r, b + 4)
#define TM_P16(r, b) TM_P8(r, b), TM_P8(r, b + 8)

// registers r[B .. B+N) -> N consecutive columns of this thread's tensor-memory lane
template <int B, int N>
__device__ __forceinline__ void tm_store(uint32_t taddr, const float (&r)[kTmMaxCnt]) {
  if constexpr (N == 16)
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                 ::"r"(taddr), TM_F16(r, B) : "memory");
  else if constexpr (N == 8)
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), TM_F8(r, B) : "memory");
  else if constexpr (N == 4)
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};" ::"r"(taddr), TM_F4(r, B) : "memory");
  else if constexpr (N == 2)
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1,%2};" ::"r"(taddr), TM_F2(r, B) : "memory");
  else
    asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), TM_F1(r, B) : "memory");
}
// N consecutive columns of this thread's tensor-memory lane -> registers r[B .. B+N)
template <int B, int N>
__device__ __forceinline__ void tm_load(float (&r)[kTmMaxCnt], uint32_t taddr) {
  if constexpr (N == 16)
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : TM_O16(r, B) : "r"(taddr) : "memory");
  else if constexpr (N == 8)
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];" : TM_O8(r, B) : "r"(taddr) : "memory");
  else if constexpr (N == 4)
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];" : TM_O4(r, B) : "r"(taddr) : "memory");
  else if constexpr (N == 2)
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : TM_O2(r, B) : "r"(taddr) : "memory");
  else
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : TM_O1(r, B) : "r"(taddr) : "memory");
}
// Waits for this thread's tensor-memory loads.  The loaded registers are named as operands so that
// no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tm_wait_loads(float (&r)[kTmMaxCnt]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : TM_P16(r, 0), TM_P16(r, 16)::"memory");
}
__device__ __forceinline__ void tm_wait_stores() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tm_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tm_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Named barrier over the 128 threads of one quadrant group.
__device__ __forceinline__ void group_sync(int id) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kTmThreads / 4) : "memory");
}
// The same barrier, returning whether `pred` held for every thread of the group.
__device__ __forceinline__ bool group_all(int id, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "r"(id), "r"(kTmThreads / 4)
      : "memory");
  return r != 0;
}

// A thread's agents sit at fixed register positions in chunks of 16, 8, 4, 2, 1, 1 (positions 0,
// 16, 24, 28, 30, 31); `mask` says which chunks are in use, so that every tensor-memory access has
// a compile-time width and every register index is static.  f(base, size, offset) is called for
// each used chunk with the chunk's offset (in agents) inside the thread's block.
template <typename F>
__device__ __forceinline__ void for_chunks(uint32_t mask, F &&f) {
  int off = 0;
  if (mask & 1u) { f(IC<0>{}, IC<16>{}, off); off += 16; }
  if (mask & 2u) { f(IC<16>{}, IC<8>{}, off); off += 8; }
  if (mask & 4u) { f(IC<24>{}, IC<4>{}, off); off += 4; }
  if (mask & 8u) { f(IC<28>{}, IC<2>{}, off); off += 2; }
  if (mask & 16u) { f(IC<30>{}, IC<1>{}, off); off += 1; }
  if (mask & 32u) { f(IC<31>{}, IC<1>{}, off); }
}
__host__ __device__ inline uint32_t chunk_mask(int cnt) {
  uint32_t m = 0;
  if (cnt >= 16) { m |= 1u; cnt -= 16; }
  if (cnt >= 8) { m |= 2u; cnt -= 8; }
  if (cnt >= 4) { m |= 4u; cnt -= 4; }
  if (cnt >= 2) { m |= 8u; cnt -= 2; }
  if (cnt >= 1) { m |= 16u; cnt -= 1; }
  if (cnt >= 1) { m |= 32u; }
  return m;
}

// acc[B..B+N) += c * r[B..B+N), two lanes per instruction where the chunk allows
template <int B, int N>
__device__ __forceinline__ void axpy_chunk(float (&acc)[kTmMaxCnt], float c, const float (&r)[kTmMaxCnt]) {
  if constexpr (N >= 2) {
    const float2 cc = make_float2(c, c);
#pragma unroll
    for (int k = 0; k < N; k += 2) {
      const float2 v = __ffma2_rn(cc, make_float2(r[B + k], r[B + k + 1]), make_float2(acc[B + k], acc[B + k + 1]));
      acc[B + k] = v.x; acc[B + k + 1] = v.y;
    }
  } else {
    acc[B] = fmaf(c, r[B], acc[B]);
  }
}

__global__ void __launch_bounds__(kTmThreads, 1)
consensus_tmem_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_y,
                      const __grid_constant__ TmemArgs p) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[4];
  __shared__ uint32_t tmem_slot;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qd = warp & 3;      // quadrant of tensor memory this warp reaches = group
  const int part = warp >> 2;   // row block inside the group
  const int bar_id = 1 + qd;
  const uint32_t tile_bytes = (uint32_t)p.n * kTmTileCols * sizeof(float);
  float *tile_x = reinterpret_cast<float *>(smem_raw + (size_t)qd * (p.has_y_in ? 2 : 1) * tile_bytes);
  float *tile_y = tile_x + (size_t)p.n * kTmTileCols;

  if (threadIdx.x == 0) {
    for (int g = 0; g < 4; ++g) mbar_init(&bars[g], 1);
    mbar_fence_init();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(&tmem_slot)), "r"((uint32_t)p.alloc_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tm_fence_before_sync();
  __syncthreads();
  tm_fence_after_sync();
  const uint32_t tbase = tmem_slot + ((uint32_t)(32 * qd) << 16);

  const int cnt = p.cnt[part];
  const uint32_t mask = chunk_mask(cnt);
  const uint32_t st_col = (uint32_t)p.stcol[part];
  const uint32_t dup = (uint32_t)p.dupoff[part];
  const int row0 = p.row0[part];
  const int rstride = p.rstride;
  const bool leader = (part == 0 && lane == 0);

  const int32_t group = (int32_t)blockIdx.x * 4 + qd;
  const int32_t group_stride = (int32_t)gridDim.x * 4;

  auto issue_load = [&](int32_t tile) {
    mbar_expect_tx(&bars[qd], p.tx_bytes);
    tma_load_2d(tile_x, &map_x, tile * kTmTileCols, 0, &bars[qd]);
    if (p.has_y_in) tma_load_2d(tile_y, &map_y, tile * kTmTileCols, 0, &bars[qd]);
  };
  if (leader && group < p.tiles) issue_load(group);

  uint32_t phase = 0;
  for (int32_t tile = group; tile < p.tiles; tile += group_stride) {
    const bool landed = mbar_wait_bounded(&bars[qd], phase, (uint32_t)p.wait_polls);
    if (!group_all(bar_id, landed)) {
      // The tile never arrived: flag it, give the transfer one more bounded chance to finish (so
      // that it does not write into shared memory after the CTA has gone) and stop this group.
      if (leader) atomicExch(p.status, 1);
      mbar_wait_bounded(&bars[qd], phase, (uint32_t)p.wait_polls);
      break;
    }
    phase ^= 1u;

    float Ih[kTmMaxCnt], Jh[kTmMaxCnt], R[kTmMaxCnt];
#pragma unroll
    for (int k = 0; k < kTmMaxCnt; ++k) Ih[k] = Jh[k] = R[k] = 0.f;
    for_chunks(mask, [&](auto B, auto N, int off) {
      const float *src = tile_x + (row0 + off * rstride) * kTmTileCols + lane;
#pragma unroll
      for (int k = 0; k < decltype(N)::value; ++k) Ih[decltype(B)::value + k] = src[k * rstride * kTmTileCols];
      if (p.has_y_in) {
        const float *srcy = tile_y + (row0 + off * rstride) * kTmTileCols + lane;
#pragma unroll
        for (int k = 0; k < decltype(N)::value; ++k) Jh[decltype(B)::value + k] = srcy[k * rstride * kTmTileCols];
      }
    });

    for (int rnd = 0; rnd < p.rounds; ++rnd) {
      const TmemRound &rd = p.rd[rnd];
      if (rd.renorm) {
        const float sI = rd.preI, sJ = rd.preJ;
#pragma unroll
        for (int k = 0; k < kTmMaxCnt; ++k) { Ih[k] *= sI; Jh[k] *= sJ; }
      }
      const uint32_t buf = tbase + (uint32_t)((rnd & 1) * p.buf_cols);
      // publish the payload of this thread's agents (twice for the block that the wrap-around reads)
      if (rd.payload) {
        for_chunks(mask, [&](auto B, auto N, int off) {
          tm_store<decltype(B)::value, decltype(N)::value>(buf + st_col + off, Jh);
          if (dup) tm_store<decltype(B)::value, decltype(N)::value>(buf + st_col + dup + off, Jh);
        });
      } else {
        for_chunks(mask, [&](auto B, auto N, int off) {
          tm_store<decltype(B)::value, decltype(N)::value>(buf + st_col + off, Ih);
          if (dup) tm_store<decltype(B)::value, decltype(N)::value>(buf + st_col + dup + off, Ih);
        });
      }
      tm_wait_stores();
      tm_fence_before_sync();
      group_sync(bar_id);
      tm_fence_after_sync();
      if (rnd == 0 && leader) {
        // every thread of the group has taken its rows out of the landing tile: prefetch the next one
        const int32_t next = tile + group_stride;
        if (next < p.tiles) issue_load(next);
      }
      const uint32_t rd_col = (uint32_t)rd.rdcol[part];
      for_chunks(mask, [&](auto B, auto N, int off) { tm_load<decltype(B)::value, decltype(N)::value>(R, buf + rd_col + off); });
      tm_wait_loads(R);
      const float cI = rd.cI, cJ = rd.cJ;
      if (rd.jcopy) {
        for_chunks(mask, [&](auto B, auto N, int) {
          axpy_chunk<decltype(B)::value, decltype(N)::value>(Ih, cI, R);
#pragma unroll
          for (int k = 0; k < decltype(N)::value; ++k) Jh[decltype(B)::value + k] = R[decltype(B)::value + k];
        });
      } else {
        for_chunks(mask, [&](auto B, auto N, int) {
          axpy_chunk<decltype(B)::value, decltype(N)::value>(Ih, cI, R);
          axpy_chunk<decltype(B)::value, decltype(N)::value>(Jh, cJ, R);
        });
      }
      // no second barrier: the next round publishes into the other buffer, and nobody can publish
      // into this one again before every thread of the group has passed the next round's barrier
    }

    // results: straight from registers, one full 128-byte line per warp and row
    const int32_t col = tile * kTmTileCols + lane;
    if (col < p.d) {
      const float oI = p.outI, oJ = p.outJ;
      const int64_t row_step = (int64_t)rstride * p.ld;
      for_chunks(mask, [&](auto B, auto N, int off) {
        float *dst = p.Xo + (int64_t)(row0 + off * rstride) * p.ld + col;
#pragma unroll
        for (int k = 0; k < decltype(N)::value; ++k) __stcs(dst + k * row_step, oI * Ih[decltype(B)::value + k]);
        if (p.has_y_out) {
          float *dsty = p.Yo + (int64_t)(row0 + off * rstride) * p.ld + col;
#pragma unroll
          for (int k = 0; k < decltype(N)::value; ++k) __stcs(dsty + k * row_step, oJ * Jh[decltype(B)::value + k]);
        }
      });
    }
  }

  tm_fence_before_sync();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"((uint32_t)p.alloc_cols)
                 : "memory");
}

// ---- host side ----------------------------------------------------------------------------------

bool consensus_tmem_supports(int32_t n, int32_t rounds) {
  return n >= 2 && n <= kTmMaxRows && rounds >= 1 && rounds <= kTmMaxRounds;
}

// Arguments are assumed validated by the caller (shapes, aliasing, alignment of X / Y and ld % 4 == 0,
// d and ld within 32 bits, Y present when the first round reads it, status word present).
// wait_polls <= 0 selects the default poll budget; tx_extra is added to the byte count the landing
// barrier is armed for (non-zero only in the test of the time-out path).
ceca_status_t consensus_tmem(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                             int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds, int32_t *status,
                             int32_t wait_polls, uint32_t tx_extra, cudaStream_t stream) {
  TmemArgs a;
  std::memset(&a, 0, sizeof(a));
  a.Xo = Xo; a.Yo = Yo; a.ld = ld; a.d = (int32_t)d; a.n = n; a.rounds = rounds;
  a.has_y_out = Yo ? 1 : 0;
  a.tiles = (int32_t)((d + kTmTileCols - 1) / kTmTileCols);
  a.status = status;
  a.wait_polls = wait_polls > 0 ? wait_polls : (int32_t)kTmWaitPolls;

  // agents -> tensor-memory columns.  2-port: one region holding agents 0..n-1 in order, cut into
  // four blocks.  1-port: even rows exchange with odd rows only, so the even rows (region 0) and
  // the odd rows (region 1) each form a region of n/2 positions cut into two blocks; in position
  // space both directions of the pairing are plain shifts.
  const bool one_port = (variant == CECA_1P);
  const int regions = one_port ? 2 : 1;
  const int len = one_port ? n / 2 : n;                 // positions per region
  const int blocks = kTmParts / regions;                // row blocks per region
  const int cb = (len + blocks - 1) / blocks;           // agents per block (the last may hold fewer)
  const int span = len + cb;                            // region + the repeated first block
  a.rstride = one_port ? 2 : 1;
  a.buf_cols = regions * span;
  int alloc = 32;
  while (alloc < 2 * a.buf_cols) alloc *= 2;
  if (alloc > 512 || cb > kTmMaxCnt) return CECA_ERR_UNSUPPORTED;
  a.alloc_cols = alloc;
  int pos0[kTmParts], region_of[kTmParts];
  for (int q = 0; q < kTmParts; ++q) {
    region_of[q] = q / blocks;
    const int b = q % blocks;
    pos0[q] = b * cb < len ? b * cb : len;
    const int c = len - pos0[q] < cb ? len - pos0[q] : cb;
    a.cnt[q] = (int16_t)c;
    a.stcol[q] = (int16_t)(region_of[q] * span + pos0[q]);
    a.dupoff[q] = (int16_t)((b == 0 && c > 0) ? len : 0);
    a.row0[q] = (int16_t)(one_port ? 2 * pos0[q] + region_of[q] : pos0[q]);
  }

  double alpha = 1.0, beta = 1.0;
  bool first_needs_y = false;
  for (int32_t t = 0; t < rounds; ++t) {
    Plan plan;
    ceca_status_t st = make_plan(n, variant, k0 + t, &plan);
    if (st != CECA_OK) return st;
    if (t == 0) first_needs_y = plan.reads_y;
    TmemRound &r = a.rd[t];
    if (t > 0 && t % kTmRenormEvery == 0) {  // fold the scales back so that the scaled values stay in range
      r.renorm = 1; r.preI = (float)alpha; r.preJ = (float)beta;
      alpha = 1.0; beta = 1.0;
    }
    const double wa = plan.rd.a, wb = plan.rd.b;
    const double zeta = plan.rd.payload ? beta : alpha;
    r.payload = (uint8_t)plan.rd.payload;
    r.cI = (float)((1.0 - wa) * zeta / (wa * alpha));
    if (plan.rd.b_num == 0) { r.jcopy = 1; r.cJ = 0.f; }
    else r.cJ = (float)((1.0 - wb) * zeta / (wb * beta));
    alpha = wa * alpha;
    beta = plan.rd.b_num == 0 ? zeta : wb * beta;
    const int hop = plan.walk.hop;
    for (int q = 0; q < kTmParts; ++q) {
      int start;
      if (!one_port) {
        start = ((pos0[q] - hop) % len + len) % len;                    // agent i receives from i - s
      } else {
        const int hh = (hop - 1) / 2;                                   // pairing offset o = 2 hh + 1
        if (region_of[q] == 0) start = span + (pos0[q] + hh) % len;     // even row 2e <- odd row 2(e+hh)+1
        else start = ((pos0[q] - hh) % len + len) % len;                // odd row 2f+1 <- even row 2(f-hh)
      }
      r.rdcol[q] = (int16_t)start;
    }
  }
  a.outI = (float)alpha; a.outJ = (float)beta;
  a.has_y_in = (Y != nullptr && first_needs_y) ? 1 : 0;
  a.tx_bytes = (uint32_t)n * kTmTileCols * sizeof(float) * (a.has_y_in ? 2u : 1u) + tx_extra;

  CUtensorMap mx, my;
  if (!tensor_map_2d(&mx, X, n, d, ld, kTmTileCols, n)) return CECA_ERR_CUDA;
  if (!tensor_map_2d(&my, a.has_y_in ? Y : X, n, d, ld, kTmTileCols, n)) return CECA_ERR_CUDA;

  constexpr size_t kMaxSmem = (size_t)4 * 2 * kTmMaxRows * kTmTileCols * sizeof(float);  // 128 KB
  static std::atomic<uint64_t> attr_done{0};
  if (set_max_shared_once(reinterpret_cast<const void *>(consensus_tmem_kernel), kMaxSmem, &attr_done) != cudaSuccess)
    return CECA_ERR_CUDA;
  const int sms = sm_count();
  if (sms <= 0) return CECA_ERR_CUDA;
  const int ctas_needed = (a.tiles + 3) / 4;
  const int grid = ctas_needed < sms ? ctas_needed : sms;
  const size_t smem = (size_t)4 * (a.has_y_in ? 2 : 1) * n * kTmTileCols * sizeof(float);
  consensus_tmem_kernel<<<grid, kTmThreads, smem, stream>>>(mx, my, a);
  return cudaGetLastError() == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

}  // namespace ceca
