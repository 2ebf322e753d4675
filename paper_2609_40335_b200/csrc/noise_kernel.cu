// Gaussian mechanism of Eq. 3 as a stand-alone pass: out[j] = scale * (out[j] + sigma*C*z_j),
// or, in fill mode, out[j] = scale * sigma*C*z_j (write only).  The stream is defined in
// noise_device.cuh.  Each thread owns one Philox counter (four consecutive elements of the
// logical row-major tensor), so the result does not depend on the launch shape.
#include <algorithm>

#include "dp_common.cuh"
#include "fma_kernels.cuh"
#include "noise_device.cuh"

namespace dpg {

namespace {

// logical tensor: rows x cols, element j = row*cols + col lives at out[row*ld + col]
template <bool kFill>
__global__ void __launch_bounds__(256)
add_noise_kernel(float* __restrict__ out, long long n, int cols, long long ld, float amp,
                 float scale, NoiseKey key) {
  const long long nq = (n + 3) >> 2;
  const bool flat = (ld == cols);
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < nq;
       q += (long long)gridDim.x * blockDim.x) {
    float z[4];
    normals4((unsigned long long)q, key, z);
    const long long j = q << 2;
    if (flat && j + 3 < n) {
      float4 v = kFill ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<float4*>(out + j);
      v.x = noised(v.x, z[0], amp, scale);
      v.y = noised(v.y, z[1], amp, scale);
      v.z = noised(v.z, z[2], amp, scale);
      v.w = noised(v.w, z[3], amp, scale);
      *reinterpret_cast<float4*>(out + j) = v;
    } else {
      for (int e = 0; e < 4 && j + e < n; ++e) {
        const long long jj = j + e;
        float* o = flat ? out + jj : out + (jj / cols) * ld + (jj % cols);
        *o = noised(kFill ? 0.f : *o, z[e], amp, scale);
      }
    }
  }
}

}  // namespace

dp_status launch_add_noise(float* out, long long rows, int cols, long long ld, bool fill, float amp,
                           float scale, uint64_t seed, uint32_t tensor_id, uint32_t step,
                           cudaStream_t st) {
  const long long n = rows * cols;
  if (n == 0) return DP_OK;
  const long long nq = (n + 3) >> 2;
  const long long want = (nq + 255) / 256;
  // Fill mode is meant to run beside another kernel (it depends on no gradient): four blocks
  // per SM leave half of every SM's thread slots free for it.
  const int grid = (int)std::min<long long>(want, (long long)sm_count() * (fill ? 4 : 16));
  const NoiseKey key{uint32_t(seed), uint32_t(seed >> 32), tensor_id, step};
  static bool carveout_set = false;
  if (fill && !carveout_set) {
    // same shared-memory carve-out as the TMA kernels, so that both can be resident on one SM
    DP_CUDA_OK(cudaFuncSetAttribute(add_noise_kernel<true>,
                                    cudaFuncAttributePreferredSharedMemoryCarveout,
                                    cudaSharedmemCarveoutMaxShared));
    carveout_set = true;
  }
  if (fill)
    add_noise_kernel<true><<<grid, 256, 0, st>>>(out, n, cols, ld, amp, scale, key);
  else
    add_noise_kernel<false><<<grid, 256, 0, st>>>(out, n, cols, ld, amp, scale, key);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
