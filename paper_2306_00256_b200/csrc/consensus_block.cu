// Fused CECA consensus rounds (Sec. 3.1 "Main recursions", Algorithm 2; the 1-port pairing of Sec. 3.2
// further down) with register-resident blocks of agents: most of every round's exchange never leaves the register file, and what the
// kernel executes per value and round is close to the one fused multiply-add it has to do.
//
// Layout.  A CTA owns one column tile of all n rows (TMA tensor loads into shared memory).  A thread
// is two adjacent matrix columns of one block of agents: LPB threads side by side cover the 2 * LPB
// columns of the tile, and each keeps I and J of a contiguous block of CB agents (rows i0 .. i0+CB-1)
// of its two columns in registers, at static register positions.  LPB = 32 (a block is a warp, 64-column
// tiles) serves n <= 150; LPB = 16 and 8 (32- and 16-column tiles, two and four blocks per warp) let
// all rows of a tile fit on one SM, two CTAs at a time up to n = 400 and n = 800, and one up to n = 1152
// (the paper's n = 1026).  Two ways of
// cutting n rows into blocks, both with compile-time trip counts for every loop over a block:
//   balanced (LPB >= 16): the first blocks hold CB agents, the others CB-1 (one predicated row);
//   uniform (LPB = 8): every block holds CB agents except the last, which holds what is left; its
//     surplus register rows ("phantom" rows, index >= n) are computed like the others but never
//     stored, and no real row ever receives from one, because sources are taken modulo n.  Threads
//     beyond the last block duplicate it (same values to the same shared-memory addresses) and
//     store nothing.  Equal block sizes are what keeps the 16-column tiles free of bank conflicts.
//
// Why this cuts the exchange.  In round r of CECA-2P agent i receives from agent i - s with
// s = n_r + delta_r, and s roughly doubles every round (1, 2, 3, 6, 12, 24, 48 for n = 97).  While
// s is smaller than a block, row offset j >= s of a block receives from offset j - s of the same
// thread: a register-to-register update with compile-time indices (one instantiation of the round
// body per value of s, selected by a uniform switch).  Only the first s rows of a block need a
// value from the previous block, so only the last s rows of every block are published in shared
// memory.  Rounds with s >= block size exchange every row.  For n = 97 (blocks of 25 agents)
// that is (1+2+3+6+12+24)/25 + 1 = 2.9 full exchanges instead of 7.  All shared-memory accesses are
// 64-bit, addressed as one base pointer plus compile-time offsets, and conflict free: half a warp
// touches 32 consecutive floats of one row (LPB >= 16), or, for LPB = 8, two 16-float row segments
// that lie CB rows apart -- CB is odd there, so the two fall into different halves of the 32 banks.
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
#include "consensus_block.cuh"

namespace ceca {

// Instantiated in consensus_block_narrow.cu and consensus_block_1p.cu.
cudaError_t launch_block_narrow(int lpb, int cb, const CUtensorMap *maps, BlockArgs &a, int threads, int cmin, bool launch,
                                int *ctas_per_sm, cudaStream_t stream);
cudaError_t launch_block_1p(int lpb, int cb, const CUtensorMap *maps, BlockArgs &a, int threads, int cmin, bool launch,
                            int *ctas_per_sm, cudaStream_t stream);

// ---- host side ----------------------------------------------------------------------------------

// Geometry by n: threads per block of agents (tile = 2 * LPB columns), number of blocks, agents per block.
//   LPB = 32 (n <= 150): blocks are warps; as few and as large as the register file allows (25 agents
//     take 100 state registers), because a round whose shift reaches the block size exchanges every
//     row through shared memory and there are about log2(blocks) such rounds; 1, 2 or a multiple of 4
//     warps, so that the warps of a CTA, which move in lockstep from barrier to barrier, load the four
//     schedulers of an SM evenly (5, 6, 7 or 9 warps measured 15-40 % slower than 4 or 8).  Twelve warps of
//     22 agents (n = 201-256) leave one CTA per SM and lose 15-20 % to 32-column tiles with two; from
//     n = 150 on eight half-warp blocks (128 threads, more CTAs per SM) are 5-9 % faster than eight warps.
//   LPB = 16 (n <= 400), LPB = 8 (n <= 1152): narrower tiles, so that all n rows of a tile (three
//     tiles' worth: landed, two exchange tiles) still fit in shared memory.  Two candidates each, and
//     the launch takes the one that puts more CTAs on an SM (the compact one on a tie):
//       `kBkCompact`: at most 256 threads (8 or 16 resp. 32 blocks of up to 25 agents), which at 128
//         registers fits two CTAs per SM where shared memory allows it too -- measured 20-35 % faster
//         than one CTA per SM (n = 350-400, 600-800), even where the 128-register form spills a little;
//       `kBkPlain`: LPB = 16: blocks of 20-23 agents, sizes whose 128-register form does not spill;
//         LPB = 8: up to 512 threads of small blocks, the best of the one-CTA-per-SM shapes measured.
//     LPB = 8 needs an odd CB (see the bank argument at the top).
struct BlockGeom {
  int lpb, cb, blocks, threads;
  int nfull;   // see BlockArgs
  int cmin;    // size of the smallest block that a partial round's source rows may lie in
};
constexpr int kBkMaxRows = 1152;
constexpr int kBkPlain = 0, kBkCompact = 1;
constexpr int kBkMaxRows1p = 416;   // CECA-1P: sixteen half-warp blocks of 26 agents
// CECA-1P: n / 2 pairs of rows in blocks of C or C - 1 pairs; cb = 2 C, cmin in pairs.  1, 2, 4 or 8
// warps on 64-column tiles up to n = 208, sixteen half-warp blocks on 32-column tiles above.
static bool block_geometry_1p(int n, BlockGeom *g) {
  if (n < 2 || (n & 1) || n > kBkMaxRows1p) return false;
  const int pairs = n / 2;
  int blocks = n <= 26 ? 1 : n <= 52 ? 2 : n <= 104 ? 4 : n <= 208 ? 8 : 16;
  if (blocks > pairs) blocks = pairs;
  const int c = (pairs + blocks - 1) / blocks;
  g->lpb = n <= 208 ? 32 : 16;
  g->blocks = blocks; g->cb = 2 * c; g->threads = (g->lpb * blocks + 31) / 32 * 32;
  g->nfull = pairs - blocks * (c - 1);
  g->cmin = g->nfull == blocks ? c : c - 1;
  return g->cb <= 26;
}
static bool block_geometry(int n, int warps_override, int kind, BlockGeom *g) {
  if (n < 2 || n > kBkMaxRows) return false;
  if (n <= 400) {
    int blocks;
    if (n <= 150) {
      if (kind != kBkPlain) return false;
      g->lpb = 32;
      blocks = n <= 25 ? 1 : n <= 50 ? 2 : n <= 100 ? 4 : 8;
      if (warps_override > 0) blocks = warps_override;
    } else {
      g->lpb = 16;
      if (kind == kBkCompact) blocks = n <= 200 ? 8 : 16;
      else blocks = ((n + 22) / 23 + 1) / 2 * 2;   // an even number of blocks of at most 23 agents: whole warps
    }
    if (blocks > n) blocks = n;
    g->blocks = blocks;
    g->cb = (n + blocks - 1) / blocks;
    g->nfull = n - blocks * (g->cb - 1);          // 1 .. blocks
    g->cmin = g->nfull == blocks ? g->cb : g->cb - 1;
  } else {
    g->lpb = 8;
    if (kind == kBkCompact) {
      g->cb = 25;   // few, roomy threads: blocks of 17-23 agents in up to 256 threads measured 15-30 % slower
      if ((n + 24) / 25 > 32) return false;   // more than 256 threads: one CTA per SM anyway
    } else {
      // one CTA per SM: many threads, the smallest size that fits in 512 of them
      static const int kSizes[] = {9, 13, 17, 21, 25};
      g->cb = 0;
      for (int cb : kSizes)
        if ((n + cb - 1) / cb <= 512 / g->lpb) { g->cb = cb; break; }
      if (!g->cb) return false;
    }
    g->blocks = (n + g->cb - 1) / g->cb;
    g->nfull = n / g->cb;
    g->cmin = g->cb;   // the sources of a partial round lie in full blocks, or are all published (last block)
  }
  if (g->cb > 25) return false;
  g->threads = (g->blocks * g->lpb + 31) / 32 * 32;
  return true;
}

struct BlockTile {
  int boxes, box_rows;
  size_t tile_bytes;
};
static BlockTile block_tile(int n, const BlockGeom &g) {
  BlockTile t;
  const int row_bytes = 2 * g.lpb * (int)sizeof(float);
  t.boxes = (n + kBkMaxBoxRows - 1) / kBkMaxBoxRows;
  t.box_rows = (n + t.boxes - 1) / t.boxes;
  if (t.boxes > 1) t.box_rows = (t.box_rows + 1) / 2 * 2;   // every box starts on a 128-byte boundary of shared memory
  int rows = t.boxes * t.box_rows;
  if (g.lpb == 8 && g.blocks * g.cb > rows) rows = g.blocks * g.cb;   // phantom rows of the last block stay inside the tile
  t.tile_bytes = ((size_t)rows * row_bytes + 127) / 128 * 128;
  return t;
}

// y_in: the first round reads Y, which takes one more shared-memory tile (at least two are needed without it).
bool consensus_block_supports(int32_t n, ceca_variant_t variant, int32_t rounds, bool y_in) {
  if (rounds < 1 || rounds > kBkMaxRounds) return false;
  if (variant == CECA_1P) {
    BlockGeom g;
    return block_geometry_1p(n, &g) && (size_t)(y_in ? 3 : 2) * block_tile(n, g).tile_bytes <= kBkSmemLimit;
  }
  if (variant != CECA_2P) return false;
  for (int kind = 0; kind < 2; ++kind) {
    BlockGeom g;
    if (block_geometry(n, 0, kind, &g) && (size_t)(y_in ? 3 : 2) * block_tile(n, g).tile_bytes <= kBkSmemLimit) return true;
  }
  return false;
}

// Fills the geometry-dependent launch arguments for candidate `kind` and either launches it or only
// reports its CTAs per SM.  CECA_ERR_UNSUPPORTED: this candidate does not exist for n or does not fit.
static ceca_status_t block_dispatch(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d, int64_t ld,
                                    BlockArgs &a, bool one_port, int kind, int warps_override, uint32_t tx_extra,
                                    bool launch, int *ctas_per_sm, cudaStream_t stream) {
  BlockGeom g;
  if (one_port ? (kind != kBkPlain || !block_geometry_1p(n, &g)) : !block_geometry(n, warps_override, kind, &g))
    return CECA_ERR_UNSUPPORTED;
  const BlockTile t = block_tile(n, g);
  if ((size_t)(a.has_y_in ? 3 : 2) * t.tile_bytes > kBkSmemLimit) return CECA_ERR_UNSUPPORTED;
  const int tile_cols = 2 * g.lpb;
  a.blocks = g.blocks; a.nfull = g.nfull; a.boxes = t.boxes; a.box_rows = t.box_rows; a.tile_bytes = (uint32_t)t.tile_bytes;
  a.tiles = (int32_t)((d + tile_cols - 1) / tile_cols);
  // a box counts in full towards the barrier, rows and columns outside the matrix included
  a.tx_bytes = (uint32_t)t.boxes * t.box_rows * tile_cols * sizeof(float) * (a.has_y_in ? 2u : 1u) + tx_extra;

  CUtensorMap maps[2];   // X in, Y in (X again when Y is not read)
  if (launch) {
    if (!tensor_map_2d(&maps[0], X, n, d, ld, tile_cols, t.box_rows)) return CECA_ERR_CUDA;
    if (!tensor_map_2d(&maps[1], a.has_y_in ? Y : X, n, d, ld, tile_cols, t.box_rows)) return CECA_ERR_CUDA;
  }

  cudaError_t e = cudaErrorInvalidConfiguration;
  if (one_port) {
    e = launch_block_1p(g.lpb, g.cb, maps, a, g.threads, g.cmin, launch, ctas_per_sm, stream);
    if (e == cudaErrorInvalidConfiguration) return CECA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
  }
#define CECA_BK_LAUNCH(CB) case CB: e = launch_block<CB, kLpb, false>(maps, a, g.threads, g.cmin, launch, ctas_per_sm, stream); break;
  if (g.lpb == 32) {
    constexpr int kLpb = 32;
    switch (g.cb) {
      CECA_BK_LAUNCH(1) CECA_BK_LAUNCH(2) CECA_BK_LAUNCH(3) CECA_BK_LAUNCH(4) CECA_BK_LAUNCH(5) CECA_BK_LAUNCH(6)
      CECA_BK_LAUNCH(7) CECA_BK_LAUNCH(8) CECA_BK_LAUNCH(9) CECA_BK_LAUNCH(10) CECA_BK_LAUNCH(11) CECA_BK_LAUNCH(12)
      CECA_BK_LAUNCH(13) CECA_BK_LAUNCH(14) CECA_BK_LAUNCH(15) CECA_BK_LAUNCH(16) CECA_BK_LAUNCH(17) CECA_BK_LAUNCH(18)
      CECA_BK_LAUNCH(19) CECA_BK_LAUNCH(20) CECA_BK_LAUNCH(21) CECA_BK_LAUNCH(22) CECA_BK_LAUNCH(23) CECA_BK_LAUNCH(24)
      CECA_BK_LAUNCH(25)
      default: break;
    }
  } else {
    e = launch_block_narrow(g.lpb, g.cb, maps, a, g.threads, g.cmin, launch, ctas_per_sm, stream);
  }
#undef CECA_BK_LAUNCH
  if (e == cudaErrorInvalidConfiguration) return CECA_ERR_UNSUPPORTED;
  return e == cudaSuccess ? CECA_OK : CECA_ERR_CUDA;
}

// Arguments are assumed validated by the caller (shapes, aliasing, 16-byte alignment of X / Y and
// ld % 4 == 0, d and ld within 32 bits, Y present when the first round reads it, status word).
// The caller has checked consensus_block_supports.  `warps_override` > 0 forces the number of
// blocks for n <= 150 (used to measure the alternatives).
ceca_status_t consensus_block(const float *X, const float *Y, float *Xo, float *Yo, int32_t n, int64_t d,
                              int64_t ld, ceca_variant_t variant, int64_t k0, int32_t rounds, int32_t *status,
                              int32_t wait_polls, uint32_t tx_extra, int warps_override, cudaStream_t stream) {
  const bool one_port = variant == CECA_1P;
  BlockArgs a;
  std::memset(&a, 0, sizeof(a));
  a.Xo = Xo; a.Yo = Yo; a.ld = ld; a.d = (int32_t)d; a.n = n; a.rounds = rounds;
  a.has_y_out = Yo ? 1 : 0;
  a.status = status;
  a.wait_polls = wait_polls > 0 ? wait_polls : (int32_t)kBkWaitPolls;

  double alpha = 1.0, beta = 1.0;
  bool first_needs_y = false;
  for (int32_t t = 0; t < rounds; ++t) {
    Plan plan;
    ceca_status_t st = make_plan(n, variant, k0 + t, &plan);
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
  if (!consensus_block_supports(n, variant, rounds, a.has_y_in != 0)) return CECA_ERR_UNSUPPORTED;

  // The candidate geometries are asked how many CTAs they put on an SM; the first of the best is launched.
  int best_kind = -1, best_ctas = 0;
  for (int kind = 1; kind >= 0; --kind) {   // the compact candidate first: it wins ties
    int ctas = 0;
    const ceca_status_t st = block_dispatch(X, Y, Xo, Yo, n, d, ld, a, one_port, kind, warps_override, tx_extra, false, &ctas, stream);
    if (st == CECA_OK && ctas > best_ctas) { best_ctas = ctas; best_kind = kind; }
    else if (st != CECA_OK && st != CECA_ERR_UNSUPPORTED) return st;
  }
  if (best_kind < 0) return CECA_ERR_UNSUPPORTED;
  int ctas = 0;
  return block_dispatch(X, Y, Xo, Yo, n, d, ld, a, one_port, best_kind, warps_override, tx_extra, true, &ctas, stream);
}

}  // namespace ceca
