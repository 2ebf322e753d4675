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
                 float scale, NoiseKey key, const uint32_t* __restrict__ step_dev, long long q0) {
  key.step = effective_step(key.step, step_dev);
  const long long nq = (n + 3) >> 2;
  const bool flat = (ld == cols);
  // 16-byte accesses only on a 16-byte aligned base (the fused entry points accept any fp32
  // tensor; an unaligned one takes the scalar branch)
  const bool vec = flat && ((reinterpret_cast<uintptr_t>(out) & 15u) == 0);
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < nq;
       q += (long long)gridDim.x * blockDim.x) {
    float z[4];
    normals4((unsigned long long)(q0 + q), key, z);       // q0: first counter of a slice
    const long long j = q << 2;
    if (vec && j + 3 < n) {
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

// Exhaustive error scan of the fp32 Box-Muller factors.  k runs over all 2^24 values of the
// 24-bit integer that feeds the factor.  out[0] = max relative error of r = sqrt(-2 ln u1) over
// the inputs with r^2 <= t_max, out[1] = max absolute error of cos / sin(2 pi u2), out[2] = the
// largest r seen, all against float64; out[3] = the r^2 threshold compiled into box_muller.
__global__ void noise_error_scan_kernel(float t_max, double* out) {
  double er = 0.0, ed = 0.0, rmax = 0.0;
  for (uint32_t k = blockIdx.x * blockDim.x + threadIdx.x; k < (1u << 24); k += gridDim.x * blockDim.x) {
    const float t = bm_t_f32(k);
    if (t <= t_max) {
      const double r32 = (double)__fsqrt_rn(t);
      const double r64 = sqrt(-2.0 * log(double(k + 1u) * 5.9604644775390625e-08));
      if (r64 > 0.0) er = fmax(er, fabs(r32 - r64) / r64);
      rmax = fmax(rmax, r64);
    }
    float s, c;
    bm_dir_f32(k, s, c);
    double s64, c64;
    sincospi(double(k) * 1.1920928955078125e-07, &s64, &c64);
    ed = fmax(ed, fmax(fabs((double)s - s64), fabs((double)c - c64)));
  }
  // block-free reduction: doubles compare as integers when non-negative
  atomicMax(reinterpret_cast<unsigned long long*>(out + 0), (unsigned long long)__double_as_longlong(er));
  atomicMax(reinterpret_cast<unsigned long long*>(out + 1), (unsigned long long)__double_as_longlong(ed));
  atomicMax(reinterpret_cast<unsigned long long*>(out + 2), (unsigned long long)__double_as_longlong(rmax));
}

}  // namespace

dp_status launch_noise_error_scan(float t_max, double* out3 /*4 doubles*/, cudaStream_t st) {
  DP_CUDA_OK(cudaMemsetAsync(out3, 0, 3 * sizeof(double), st));
  if (t_max <= 0.f) t_max = DPG_NOISE_TAIL_T;             // scan exactly the fp32 path in use
  noise_error_scan_kernel<<<sm_count() * 8, 256, 0, st>>>(t_max, out3);
  DP_LAUNCH_OK();
  const double thr = DPG_NOISE_TAIL_T;
  DP_CUDA_OK(cudaMemcpyAsync(out3 + 3, &thr, sizeof(double), cudaMemcpyHostToDevice, st));
  return DP_OK;
}

dp_status launch_add_noise(float* out, long long rows, int cols, long long ld, bool fill, float amp,
                           float scale, uint64_t seed, uint32_t tensor_id, uint32_t step,
                           cudaStream_t st, long long first_quad) {
  const long long n = rows * cols;
  if (n == 0) return DP_OK;
  const long long nq = (n + 3) >> 2;
  const long long want = (nq + 255) / 256;
  // Fill mode is meant to run beside another kernel (it depends on no gradient): four blocks
  // per SM leave half of every SM's thread slots free for it.
  const int grid = (int)std::min<long long>(want, (long long)sm_count() * (fill ? 4 : 16));
  const NoiseKey key{uint32_t(seed), uint32_t(seed >> 32), tensor_id, step};
  if (fill && first_use_on_this_device(reinterpret_cast<const void*>(&launch_add_noise))) {
    // same shared-memory carve-out as the TMA kernels, so that both can be resident on one SM
    DP_CUDA_OK(cudaFuncSetAttribute(add_noise_kernel<true>,
                                    cudaFuncAttributePreferredSharedMemoryCarveout,
                                    cudaSharedmemCarveoutMaxShared));
  }
  if (fill)
    add_noise_kernel<true><<<grid, 256, 0, st>>>(out, n, cols, ld, amp, scale, key, g_step_dev, first_quad);
  else
    add_noise_kernel<false><<<grid, 256, 0, st>>>(out, n, cols, ld, amp, scale, key, g_step_dev, first_quad);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
