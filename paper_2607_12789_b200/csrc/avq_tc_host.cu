// Host-side helpers of the tensor-core path: driver entry point for tensor-map encoding.
#include <mutex>

#include "avq_tc_common.cuh"

namespace avq {
namespace tc {

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

namespace {
// Encoding a tensor map costs a few microseconds of host time and a forward needs seven of them, so
// recent encodings are kept: the result depends only on (base, rank, dims, box).
struct TmapKey {
  const void* base;
  int rank;
  uint64_t dims[3];
  uint32_t box[3];
  bool operator==(const TmapKey& o) const {
    if (base != o.base || rank != o.rank) return false;
    for (int i = 0; i < 3; ++i)
      if (dims[i] != o.dims[i] || box[i] != o.box[i]) return false;
    return true;
  }
};
constexpr int kTmapCache = 128;
std::mutex g_tmap_mu;
TmapKey g_tmap_keys[kTmapCache];
CUtensorMap g_tmap_vals[kTmapCache];
int g_tmap_used = 0, g_tmap_next = 0;
}  // namespace

avq_status make_tmap_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                          const uint32_t* box) {
  if (rank < 1 || rank > 3) return AVQ_ERR_UNSUPPORTED;
  TmapKey key = {};
  key.base = base;
  key.rank = rank;
  for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  {
    std::lock_guard<std::mutex> lock(g_tmap_mu);
    for (int i = 0; i < g_tmap_used; ++i)
      if (g_tmap_keys[i] == key) { *map = g_tmap_vals[i]; return AVQ_OK; }
  }
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return AVQ_ERR_CUDA;
  cuuint64_t gdim[5];
  cuuint64_t gstride[4];
  cuuint32_t bdim[5], estr[5];
  uint64_t pitch = 2;
  for (int i = 0; i < rank; ++i) {
    gdim[i] = dims[i];
    bdim[i] = box[i];
    estr[i] = 1;
    pitch *= dims[i];
    if (i + 1 < rank) gstride[i] = pitch;   // byte stride of dimension i+1
  }
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim,
                  gstride, bdim, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return AVQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_tmap_mu);
  const int slot = g_tmap_used < kTmapCache ? g_tmap_used++ : (g_tmap_next++ % kTmapCache);
  g_tmap_keys[slot] = key;
  g_tmap_vals[slot] = *map;
  return AVQ_OK;
}

}  // namespace tc
}  // namespace avq
