// TMA tensor-map construction on the host.
#include "tma_host.cuh"

#include <cstring>
#include <mutex>
#include <unordered_map>

namespace dpg {

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Encoded maps are kept: a tensor map is a pure function of (address, pitch, extents, box), so
// a step that is issued call by call every iteration (no CUDA graph) pays the driver's encode
// once per tensor instead of once per call.  Bounded: the table is cleared when it is full.
struct TmapKey {
  const void* base; int64_t ld; int cols, rows, batch, box_cols, box_rows;
  bool operator==(const TmapKey& o) const {
    return base == o.base && ld == o.ld && cols == o.cols && rows == o.rows && batch == o.batch &&
           box_cols == o.box_cols && box_rows == o.box_rows;
  }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey& k) const {
    uint64_t h = reinterpret_cast<uint64_t>(k.base) * 0x9E3779B97F4A7C15ull;
    auto mix = [&](uint64_t v) { h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2); };
    mix(uint64_t(k.ld)); mix(uint64_t(k.cols) << 32 | uint32_t(k.rows));
    mix(uint64_t(k.batch) << 32 | uint32_t(k.box_cols) << 16 | uint32_t(k.box_rows));
    return size_t(h);
  }
};
constexpr size_t kTmapCacheMax = 4096;
std::mutex g_tmap_mutex;
std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> g_tmap_cache;
long long g_tmap_encodes = 0;
}  // namespace

long long tmap_encode_count() { return g_tmap_encodes; }

dp_status make_tmap_bf16_3d(CUtensorMap* out, const void* base, int64_t ld, int cols, int rows,
                            int batch, int box_cols, int box_rows) {
  const TmapKey key{base, ld, cols, rows, batch, box_cols, box_rows};
  {
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    auto it = g_tmap_cache.find(key);
    if (it != g_tmap_cache.end()) { memcpy(out, &it->second, sizeof(CUtensorMap)); return DP_OK; }
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) { g_last_cuda_error = (int)cudaErrorSymbolNotFound; return DP_ERR_CUDA; }
  if (!aligned16(base) || (ld % 8) != 0) return DP_ERR_ALIGNMENT;
  const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
  const cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)ld * 2 * (cuuint64_t)rows};
  const cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return DP_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_tmap_mutex);
  ++g_tmap_encodes;
  if (g_tmap_cache.size() >= kTmapCacheMax) g_tmap_cache.clear();
  g_tmap_cache.emplace(key, *out);
  return DP_OK;
}

}  // namespace dpg
