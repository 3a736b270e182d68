// Host-side helper: tensor maps over a channel-sliced activation tensor, encoded through the
// driver entry point (looked up at run time, so the library does not link against libcuda).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

namespace gi {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn tensor_map_encoder() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  });
  return fn;
}

// 2-D map over [slices][pixels] of 8-byte pixel-slices (4 fp16 channels): a box of box_px pixels x
// box_slices slices lands in shared memory as box_slices rows of box_px * 8 contiguous bytes;
// pixels and slices outside the tensor read as zeros.  box_px <= 256, an even pixel start keeps
// the copy 16-byte aligned.  Returns a cudaError_t as int.
inline int encode_plane_map(CUtensorMap* map, const void* base, unsigned long long total_px, int n_slices, int box_px,
                            int box_slices) {
  EncodeTiledFn enc = tensor_map_encoder();
  if (!enc) return static_cast<int>(cudaErrorNotSupported);
  const cuuint64_t gdim[2] = {total_px, static_cast<cuuint64_t>(n_slices)};
  const cuuint64_t gstride[1] = {total_px * 8u};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_px), static_cast<cuuint32_t>(box_slices)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult cr = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return cr == CUDA_SUCCESS ? 0 : static_cast<int>(cudaErrorInvalidValue);
}

// Tensor maps depend on device addresses: one cached entry per launch of an executable, kept in
// a cache the executable owns through an opaque pointer.
struct MapEntry {
  const void* in = nullptr;
  CUtensorMap map;
};
struct MapCache {
  std::vector<MapEntry> maps;
};
inline MapEntry& map_cache_entry(void** state, int launch_index) {
  if (!*state) *state = new MapCache();
  MapCache* c = static_cast<MapCache*>(*state);
  if (c->maps.size() <= static_cast<size_t>(launch_index)) c->maps.resize(launch_index + 1);
  return c->maps[launch_index];
}
inline void map_cache_release(void* state) { delete static_cast<MapCache*>(state); }

}  // namespace gi
