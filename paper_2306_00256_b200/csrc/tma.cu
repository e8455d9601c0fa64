// Host helpers of the fused consensus kernels: encoded tensor maps (cached) and device properties.
#include "tma.h"

#include <atomic>
#include <mutex>

namespace ceca {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime's driver entry point query (no link against libcuda).
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

namespace {
struct MapKey {
  const float *base;
  int64_t d, ld;
  int32_t n, tile_cols, box_rows;
  bool operator==(const MapKey &o) const {
    return base == o.base && d == o.d && ld == o.ld && n == o.n && tile_cols == o.tile_cols && box_rows == o.box_rows;
  }
};
constexpr int kMapCacheSlots = 32;
struct MapCache {
  std::mutex mutex;
  MapKey keys[kMapCacheSlots];
  CUtensorMap maps[kMapCacheSlots];
  bool used[kMapCacheSlots] = {};
  int next = 0;  // round-robin replacement
};
MapCache g_maps;
}  // namespace

bool tensor_map_2d(CUtensorMap *map, const float *base, int32_t n, int64_t d, int64_t ld, int tile_cols,
                   int box_rows) {
  const MapKey key{base, d, ld, n, tile_cols, box_rows};
  std::lock_guard<std::mutex> lock(g_maps.mutex);
  for (int s = 0; s < kMapCacheSlots; ++s)
    if (g_maps.used[s] && g_maps.keys[s] == key) {
      *map = g_maps.maps[s];
      return true;
    }
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)n};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)tile_cols, (cuuint32_t)box_rows};
  const cuuint32_t elem[2] = {1, 1};
  if (enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, elem,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  const int s = g_maps.next;
  g_maps.next = (s + 1) % kMapCacheSlots;
  g_maps.keys[s] = key;
  g_maps.maps[s] = *map;
  g_maps.used[s] = true;
  return true;
}

int sm_count() {
  constexpr int kMaxDevices = 64;
  static std::atomic<int> cached[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 0;
  if (dev < kMaxDevices) {
    const int c = cached[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (dev < kMaxDevices) cached[dev].store(sms, std::memory_order_relaxed);
  return sms;
}

cudaError_t set_max_shared_once(const void *kernel, size_t bytes, std::atomic<uint64_t> *done_mask) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && (done_mask->load(std::memory_order_acquire) >> dev & 1u)) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  if (tracked) done_mask->fetch_or((uint64_t)1 << dev, std::memory_order_release);
  return cudaSuccess;
}

}  // namespace ceca
