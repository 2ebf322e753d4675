// fp32 operands on the bf16 tensor cores: every fp32 value x is split into two bf16 terms,
//   hi = bf16(x),  lo = bf16(x - hi),   x = hi + lo up to 2^-17 |x|,
// and a product x*y is taken as hi*hi' + hi*lo' + lo*hi' (the dropped lo*lo' is below 2^-16 of the
// product) -- three tensor-core products with fp32 accumulation instead of one, the same idea as
// the "3 x TF32" scheme with 16 instead of 21 mantissa bits, far inside the 1e-4 the fp32 path has
// to meet, and at three bf16 MMAs cheaper than three TF32 MMAs (which run at half the bf16 rate).
//
// The three products become ONE ordinary product of two widened operands, so the bf16 kernels
// run unchanged:
//   contraction over columns (the Gram matrices of the ghost norm):
//       X = [hi | hi | lo],  Y = [hi | lo | hi]   ->  X Y^T = hi hi^T + hi lo^T + lo hi^T
//   contraction over tokens (G^T A of the clipped sum and of the DIRECT norm): per example
//       G' = [hi ; hi ; lo] (3T rows),  A' = [hi ; lo ; hi]   ->  G'^T A' = the three products.
// For the clipped sum the clip factor R_i (Eq. 7) multiplies G in fp32 BEFORE the split, so the
// GEMM itself runs unscaled and no bf16 rounding of R_i * g occurs.
#include <cuda_bf16.h>

#include <algorithm>

#include "dp_common.cuh"
#include "split_kernels.cuh"

namespace dpg {

namespace {

__device__ __forceinline__ void split2(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// X, Y: (rows, 3*cp) bf16; column blocks of width cp (c rounded up to 8; the padding is zero)
__global__ void __launch_bounds__(256)
split_cols_kernel(const float* __restrict__ src, long long lds, long long rows, int c, int cp,
                  __nv_bfloat16* __restrict__ X, __nv_bfloat16* __restrict__ Y) {
  const long long total = rows * cp;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / cp;
    const int col = int(e - r * cp);
    __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi;
    if (col < c) split2(src[r * lds + col], hi, lo);
    __nv_bfloat16* x = X + r * 3 * cp + col;
    __nv_bfloat16* y = Y + r * 3 * cp + col;
    x[0] = hi; x[cp] = hi; x[2 * cp] = lo;
    y[0] = hi; y[cp] = lo; y[2 * cp] = hi;
  }
}

// dst: (B, 3T, cp) bf16: rows [0,T) / [T,2T) / [2T,3T) of example i hold the three terms
// {hi,hi,lo} (lo_slab = 2) or {hi,lo,hi} (lo_slab = 1) of scale[i] * src[i]
__global__ void __launch_bounds__(256)
split_rows_kernel(const float* __restrict__ src, long long lds, int B, int T, int c, int cp,
                  const float* __restrict__ scale, int lo_slab, __nv_bfloat16* __restrict__ dst) {
  const long long total = (long long)B * T * cp;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / cp;                   // token row i*T + t
    const int col = int(e - r * cp);
    const int i = int(r / T), t = int(r - (long long)i * T);
    __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi;
    if (col < c) split2(src[r * lds + col] * (scale ? scale[i] : 1.f), hi, lo);
    __nv_bfloat16* d0 = dst + ((long long)i * 3 * T + t) * cp + col;
#pragma unroll
    for (int sl = 0; sl < 3; ++sl) d0[(long long)sl * T * cp] = (sl == lo_slab) ? lo : hi;
  }
}

int grid_for(long long total) {
  return (int)std::min<long long>((total + 255) / 256, (long long)sm_count() * 16);
}

}  // namespace

dp_status launch_split_cols(const float* src, int64_t lds, int64_t rows, int c, void* X, void* Y,
                            cudaStream_t st) {
  const int cp = split_padded(c);
  split_cols_kernel<<<grid_for(rows * cp), 256, 0, st>>>(src, lds, rows, c, cp,
                                                       static_cast<__nv_bfloat16*>(X),
                                                       static_cast<__nv_bfloat16*>(Y));
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_split_rows(const float* src, int64_t lds, int B, int T, int c, const float* scale,
                            int lo_slab, void* dst, cudaStream_t st) {
  const int cp = split_padded(c);
  split_rows_kernel<<<grid_for((long long)B * T * cp), 256, 0, st>>>(
      src, lds, B, T, c, cp, scale, lo_slab, static_cast<__nv_bfloat16*>(dst));
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
