// dp_embed_norms_static: the embedding ghost norm for callers that may not allocate.
//
// Some hosts of this library cannot hand it a workspace: code running under an allocator that
// is frozen for the duration of a step (a captured or pre-planned memory pool), plug-ins that
// are only given their input and output tensors, or bring-up code on a device whose memory is
// already fully committed.  For them the scratch of the embedding norm (one partial sum per
// example and 256-column slab) lives in a fixed array inside the library image instead of a
// caller buffer.  Nothing here calls cudaMalloc, cudaFree or any other allocating routine.
#include <mutex>

#include "dp_common.cuh"
#include "fma_kernels.cuh"

namespace dpg {
namespace {

// 64 KiB per device that loads the library, held until the process exits.
constexpr int kStaticScratchFloats = DP_STATIC_SCRATCH_FLOATS;
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// In host code `g_static_scratch` is only a handle for the runtime, not a device address:
// resolve it once per device (with that device current) and cache the result.
dp_status static_scratch_for_current_device(float** out) {
  int dev = 0;
  DP_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return DP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    DP_CUDA_OK(cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch));
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return DP_OK;
}

}  // namespace
}  // namespace dpg

using namespace dpg;

extern "C" dp_status dp_embed_norms_static(const int32_t* ids, const void* G, int64_t ldg,
                                           dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t V,
                                           float* sq, int32_t* first_occ, int32_t* dev_status,
                                           void* stream) {
  if (!ids || !G || !sq || B <= 0 || T <= 0 || d <= 0 || V <= 0 || ldg < d) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  if (T > kEmbedMaxT) return DP_ERR_UNSUPPORTED;
  const int slabs = ceil_div(d, kEmbedColsPerBlock);
  if ((long long)B * slabs > kStaticScratchFloats) return DP_ERR_SCRATCH_LIMIT;
  float* partials = nullptr;
  dp_status s = static_scratch_for_current_device(&partials);
  if (s != DP_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  // every partial that is read below is written first by the norm kernel, so the array's
  // previous contents never matter and nothing has to be cleared
  s = launch_embed_norms(ids, G, ldg, dt, B, T, d, V, partials, first_occ, dev_status, st);
  if (s != DP_OK) return s;
  return launch_reduce_partials(partials, slabs, B, sq, 1.f, nullptr, st);
}
