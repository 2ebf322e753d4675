// Shared host/device helpers of the DP-SGD hot-path library (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dp_ghost.h"

namespace dpg {

// last CUDA error code seen by an entry point (returned by dp_last_cuda_error)
extern int g_last_cuda_error;
extern int g_force_fma;
extern long long g_kernel_launches;   // kernels enqueued by this library since load

inline dp_status cuda_fail(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return DP_ERR_CUDA;
}

#define DP_CUDA_OK(expr)                                  \
  do {                                                    \
    cudaError_t _e = (expr);                              \
    if (_e != cudaSuccess) return ::dpg::cuda_fail(_e);   \
  } while (0)

#define DP_LAUNCH_OK()                                    \
  do {                                                    \
    cudaError_t _e = cudaGetLastError();                  \
    if (_e != cudaSuccess) return ::dpg::cuda_fail(_e);   \
    ++::dpg::g_kernel_launches;                           \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// number of SMs of the current device (cached per process)
int sm_count();

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
  return __bfloat162float(v);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Deterministic block-wide sum; result valid in thread 0. `red` holds >= 32 floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float r = 0.f;
  if (w == 0) {
    r = (lane < nw) ? red[lane] : 0.f;
    r = warp_sum(r);
  }
  return r;
}

// clip coefficient of Eq. 7 from a squared norm, IEEE sqrt and divide
__device__ __forceinline__ float clip_from_sq(float sq, float C) {
  const float nrm = __fsqrt_rn(sq);
  return nrm > 0.f ? fminf(1.f, __fdiv_rn(C, nrm)) : 1.f;
}

// ---- launchers implemented across the .cu files (all enqueue on `st`, no sync) ----
// sq[i] += factor * sum_j partials[i*n_per + j] (fixed order); plain_out[i] = that sum if given
dp_status launch_reduce_partials(const float* partials, int n_per, int B, float* sq,
                                 float factor, float* plain_out, cudaStream_t st);

}  // namespace dpg
