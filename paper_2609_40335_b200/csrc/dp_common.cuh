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
extern long long g_kernel_launches;
extern const uint32_t* g_step_dev;   // device counter added to every noise step (NULL: none)
extern int g_ghost_single;           // test knob: keep the single-CTA Gram kernel for T > 128
extern long long g_wait_limit;       // cycles a device-side barrier wait may take (test knob)   // kernels enqueued by this library since load

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

// number of SMs of the current device (cached per device)
int sm_count();

// One-time set-up that CUDA keeps PER DEVICE (function attributes such as the dynamic
// shared-memory limit): true the first time `key` is seen with the current device, false
// afterwards.  A process that drives several GPUs gets the set-up on each of them.
bool first_use_on_this_device(const void* key);

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

// 8 consecutive columns of one row as floats; `nvalid` columns exist, `vec` says the 16-byte
// (bf16) / 2 x 16-byte (fp32) vector path is aligned.
template <typename T>
__device__ __forceinline__ void load8(const T* p, int nvalid, bool vec, float (&v)[8]);

template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, int nvalid, bool vec,
                                                     float (&v)[8]) {
  if (vec && nvalid >= 8) {
    const uint4 q = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[2 * e] = __uint_as_float(w[e] << 16);
      v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = e < nvalid ? __bfloat162float(p[e]) : 0.f;
  }
}

template <>
__device__ __forceinline__ void load8<float>(const float* p, int nvalid, bool vec, float (&v)[8]) {
  if (vec && nvalid >= 8) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = e < nvalid ? p[e] : 0.f;
  }
}

// Clip coefficient of Eq. 7 from a squared norm, IEEE sqrt and divide.  A zero norm gives 1
// (nothing to clip).  The tied norm in + out + 2 cross can round to a tiny negative number when
// the true norm is ~0: that is clamped to zero.  A squared norm that is not finite (NaN or inf
// from corrupted inputs) gives 0 -- the example is dropped from the sum rather than added
// unclipped, so a bad norm can never break the sensitivity bound of Eq. 2.
__device__ __forceinline__ float clip_from_sq(float sq, float C) {
  if (!(fabsf(sq) <= 3.402823466e38f)) return 0.f;       // NaN or +-inf
  const float nrm = __fsqrt_rn(fmaxf(sq, 0.f));
  return nrm > 0.f ? fminf(1.f, __fdiv_rn(C, nrm)) : 1.f;
}

// ---- checked build ------------------------------------------------------------------------
// Compiled with -DDP_BOUNDS_CHECK (python -m paper_2609_40335_b200.build --check, which writes
// libdp_ghost_check.so), every index that a kernel COMPUTES from data -- a gathered column, a
// sorted position, a rank, a partial-sum slot -- is compared with the extent of the array it
// addresses before the access; an index outside ORs DP_DEV_BOUNDS into dev_status and the access
// is skipped.  It stands in for a memory checker on machines where none may be run.  In the
// normal build the test costs nothing.
#ifdef DP_BOUNDS_CHECK
__device__ __forceinline__ bool dp_in_range(long long idx, long long n, int* dev_status) {
  if (idx >= 0 && idx < n) return true;
  if (dev_status) atomicOr(dev_status, DP_DEV_BOUNDS);
  return false;
}
constexpr int kBoundsChecked = 1;
#else
__device__ __forceinline__ bool dp_in_range(long long, long long, int*) { return true; }
constexpr int kBoundsChecked = 0;
#endif

// ---- launchers implemented across the .cu files (all enqueue on `st`, no sync) ----
// sq[i] += factor * sum_j partials[i*n_per + j] (fixed order); plain_out[i] = that sum if given
dp_status launch_reduce_partials(const float* partials, int n_per, int B, float* sq,
                                 float factor, float* plain_out, cudaStream_t st);

}  // namespace dpg
