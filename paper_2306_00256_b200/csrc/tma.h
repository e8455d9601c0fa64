// Internal: mbarrier / TMA wrappers (inline PTX) shared by the fused consensus kernels, and the
// host-side cache of encoded tensor maps.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

namespace ceca {

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
// Single-CTA tensor load (no multicast): the destination is this CTA's own shared memory.
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
#endif  // __CUDACC__

// The tensor map of an n x d fp32 matrix with row pitch ld (elements), boxed as box_rows rows x
// tile_cols columns, out-of-range elements reading as zero.  Encoded maps are kept in a small
// per-process cache keyed on every argument, so that a caller that reuses its buffers pays for the
// driver's encoding once; the map only describes addresses and shapes, so an entry stays valid
// as long as the key matches.  Returns false when the driver refuses to encode.
bool tensor_map_2d(CUtensorMap *map, const float *base, int32_t n, int64_t d, int64_t ld, int tile_cols,
                   int box_rows);

// Number of SMs of the current device (cached per device ordinal); 0 on error.
int sm_count();

// Raises a kernel's dynamic shared-memory limit to `bytes` (its largest launch) and asks for the
// largest shared-memory carve-out, once per device: `done_mask` has one bit per device ordinal.
// The value never changes afterwards, so concurrent launches from several host threads cannot see
// a limit lower than the one they need.
cudaError_t set_max_shared_once(const void *kernel, size_t bytes, std::atomic<uint64_t> *done_mask);

}  // namespace ceca
