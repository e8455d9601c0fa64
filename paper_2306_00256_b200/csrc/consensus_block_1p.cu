// Register-block fused consensus (see consensus_block.cu): the CECA-1P instantiations -- blocks of an even
// number of agents, warps on 64-column tiles up to n = 208, half-warp blocks on 32-column tiles up to n = 416.
#include "consensus_block.cuh"

namespace ceca {

cudaError_t launch_block_1p(int lpb, int cb, const CUtensorMap *maps, BlockArgs &a, int threads, int cmin, bool launch,
                            int *ctas_per_sm, cudaStream_t stream) {
  cudaError_t e = cudaErrorInvalidConfiguration;
#define CECA_BK_LAUNCH(CB) case CB: e = launch_block<CB, kLpb, true>(maps, a, threads, cmin, launch, ctas_per_sm, stream); break;
  if (lpb == 32) {
    constexpr int kLpb = 32;
    switch (cb) {
      CECA_BK_LAUNCH(2) CECA_BK_LAUNCH(4) CECA_BK_LAUNCH(6) CECA_BK_LAUNCH(8) CECA_BK_LAUNCH(10) CECA_BK_LAUNCH(12)
      CECA_BK_LAUNCH(14) CECA_BK_LAUNCH(16) CECA_BK_LAUNCH(18) CECA_BK_LAUNCH(20) CECA_BK_LAUNCH(22) CECA_BK_LAUNCH(24)
      CECA_BK_LAUNCH(26)
      default: break;
    }
  } else if (lpb == 16) {
    constexpr int kLpb = 16;
    switch (cb) {   // n = 210 .. 416 in sixteen blocks
      CECA_BK_LAUNCH(14) CECA_BK_LAUNCH(16) CECA_BK_LAUNCH(18) CECA_BK_LAUNCH(20) CECA_BK_LAUNCH(22) CECA_BK_LAUNCH(24)
      CECA_BK_LAUNCH(26)
      default: break;
    }
  }
#undef CECA_BK_LAUNCH
  return e;
}

}  // namespace ceca
