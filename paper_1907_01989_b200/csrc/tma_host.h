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

// Tensor maps depend on device addresses.  The cache an executable owns (through an opaque pointer) keeps, per
// launch, the maps of the last few distinct input addresses: a caller that alternates between two arenas or two
// input buffers (a two-slot pipeline, gi_run followed by gi_run_static) encodes each map once, not on every call.
// Host threads may run one executable at the same time (with different arenas): the cache is guarded by a
// mutex and a launcher works on its own copy of the map, never on the cached one.
constexpr int kMapWays = 4;
struct MapSlot {
  const void* in[kMapWays] = {};
  CUtensorMap map[kMapWays];
  int used = 0, next = 0;
};
struct MapCache {
  std::mutex mu;
  std::vector<MapSlot> slots;
};
inline MapCache* map_cache(void** state) {
  static std::mutex create_mu;
  std::lock_guard<std::mutex> lock(create_mu);
  if (!*state) *state = new MapCache();
  return static_cast<MapCache*>(*state);
}
// Copies the map for (launch, input address) into *out, encoding it with `encode(CUtensorMap*) -> int` (a
// cudaError_t, 0 on success) if it is not cached.  Returns that error code.
template <typename Encode>
inline int map_cache_lookup(void** state, int launch_index, const void* in, CUtensorMap* out, Encode&& encode) {
  MapCache* c = map_cache(state);
  std::lock_guard<std::mutex> lock(c->mu);
  if (c->slots.size() <= static_cast<size_t>(launch_index)) c->slots.resize(launch_index + 1);
  MapSlot& s = c->slots[launch_index];
  for (int i = 0; i < s.used; ++i)
    if (s.in[i] == in) {
      *out = s.map[i];
      return 0;
    }
  int way;
  if (s.used < kMapWays) {
    way = s.used;
  } else {
    way = s.next;
    s.next = (s.next + 1) % kMapWays;
  }
  const int err = encode(&s.map[way]);
  if (err != 0) {
    if (way < s.used) s.in[way] = nullptr;  // the overwritten entry is gone
    return err;
  }
  if (way == s.used) ++s.used;
  s.in[way] = in;
  *out = s.map[way];
  return 0;
}
inline void map_cache_release(void* state) { delete static_cast<MapCache*>(state); }

}  // namespace gi
