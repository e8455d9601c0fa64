// Register-block fused consensus (see consensus_block.cu): the CECA-2P instantiations for tiles narrower
// than 64 columns -- blocks of 16 threads (n = 151 .. 400) and of 8 threads (n = 401 .. 1152).
#include "consensus_block.cuh"

namespace ceca {

cudaError_t launch_block_narrow(int lpb, int cb, const CUtensorMap *maps, BlockArgs &a, int threads, int cmin, bool launch,
                                int *ctas_per_sm, cudaStream_t stream) {
  cudaError_t e = cudaErrorInvalidConfiguration;
#define CECA_BK_LAUNCH(CB) case CB: e = launch_block<CB, kLpb, false>(maps, a, threads, cmin, launch, ctas_per_sm, stream); break;
  if (lpb == 16) {
    constexpr int kLpb = 16;
    switch (cb) {   // 8 or 16 blocks of 13 to 25 agents, or 8 to 18 blocks of 19 to 23
      CECA_BK_LAUNCH(13) CECA_BK_LAUNCH(14) CECA_BK_LAUNCH(15) CECA_BK_LAUNCH(16) CECA_BK_LAUNCH(17) CECA_BK_LAUNCH(18)
      CECA_BK_LAUNCH(19) CECA_BK_LAUNCH(20) CECA_BK_LAUNCH(21) CECA_BK_LAUNCH(22) CECA_BK_LAUNCH(23) CECA_BK_LAUNCH(24)
      CECA_BK_LAUNCH(25)
      default: break;
    }
  } else if (lpb == 8) {
    constexpr int kLpb = 8;
    switch (cb) {   // odd sizes
      CECA_BK_LAUNCH(9) CECA_BK_LAUNCH(13) CECA_BK_LAUNCH(17) CECA_BK_LAUNCH(21) CECA_BK_LAUNCH(25)
      default: break;
    }
  }
#undef CECA_BK_LAUNCH
  return e;
}

}  // namespace ceca
