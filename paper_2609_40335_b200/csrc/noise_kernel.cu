// Gaussian mechanism of Eq. 3: out[j] = scale * (out[j] + sigma*C*z_j), z ~ N(0, I).
//
// z_j is a pure function of (seed, tensor_id, step, j): Philox4x32 with 10 rounds, key =
// (seed low, seed high), counter = (j/4 low, j/4 high, tensor_id, step); the four output
// words give four normals by Box-Muller on the word pairs (x0,x1) and (x2,x3):
//   u1 = ((xa >> 8) + 1) * 2^-24 in (0,1],  u2 = (xb >> 8) * 2^-24 in [0,1)   (exact in fp32)
//   r = sqrt(-2 ln u1),  z = r cos(2 pi u2),  r sin(2 pi u2).
// Each thread owns one counter (four consecutive elements), so the result does not depend on
// the launch shape.
//
// Accuracy: fp32 logf / sqrtf / sincospif give a relative error of at most about 2.5 ulp
// (3e-7) on z, i.e. below 1e-6 absolute while r <= 3.3.  Pairs with a larger radius (0.4 % of
// them) take a float64 path, whose only error is the final rounding to fp32.
#include "dp_common.cuh"
#include "fma_kernels.cuh"

namespace dpg {

namespace {

struct U4 { uint32_t x, y, z, w; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return U4{c0, c1, c2, c3};
}

constexpr float kTailR2 = 10.89f;   // r = 3.3

__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& za, float& zb) {
  const float u1 = float((xa >> 8) + 1u) * 5.9604644775390625e-08f;   // 2^-24
  const float u2x2 = float(xb >> 8) * 1.1920928955078125e-07f;        // 2 * u2, exact
  const float t = -2.0f * logf(u1);
  if (t <= kTailR2) {
    const float r = __fsqrt_rn(t);
    float s, c;
    sincospif(u2x2, &s, &c);
    za = r * c;
    zb = r * s;
  } else {
    const double r = sqrt(-2.0 * log(double((xa >> 8) + 1u) * 5.9604644775390625e-08));
    double s, c;
    sincospi(double(xb >> 8) * 1.1920928955078125e-07, &s, &c);
    za = float(r * c);
    zb = float(r * s);
  }
}

__global__ void __launch_bounds__(256)
add_noise_kernel(float* __restrict__ out, long long n, float amp, float scale, uint32_t k0,
                 uint32_t k1, uint32_t tensor_id, uint32_t step) {
  const long long nq = (n + 3) >> 2;
  for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < nq;
       q += (long long)gridDim.x * blockDim.x) {
    const U4 x = philox4x32_10(uint32_t(q), uint32_t(uint64_t(q) >> 32), tensor_id, step, k0, k1);
    float z[4];
    box_muller(x.x, x.y, z[0], z[1]);
    box_muller(x.z, x.w, z[2], z[3]);
    const long long j = q << 2;
    if (j + 3 < n) {
      float4 v = *reinterpret_cast<float4*>(out + j);
      v.x = scale * fmaf(amp, z[0], v.x);
      v.y = scale * fmaf(amp, z[1], v.y);
      v.z = scale * fmaf(amp, z[2], v.z);
      v.w = scale * fmaf(amp, z[3], v.w);
      *reinterpret_cast<float4*>(out + j) = v;
    } else {
      for (int e = 0; e < 4 && j + e < n; ++e) out[j + e] = scale * fmaf(amp, z[e], out[j + e]);
    }
  }
}

}  // namespace

dp_status launch_add_noise(float* out, long long n, float amp, float scale, uint64_t seed,
                           uint32_t tensor_id, uint32_t step, cudaStream_t st) {
  if (n == 0) return DP_OK;
  const long long nq = (n + 3) >> 2;
  const long long want = (nq + 255) / 256;
  const int grid = (int)std::min<long long>(want, (long long)sm_count() * 16);
  add_noise_kernel<<<grid, 256, 0, st>>>(out, n, amp, scale, uint32_t(seed), uint32_t(seed >> 32),
                                         tensor_id, step);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
