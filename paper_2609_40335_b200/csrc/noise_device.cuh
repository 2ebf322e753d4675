// Device-side Gaussian stream shared by the stand-alone noise kernel and the GEMM epilogue.
//
// z_j is a pure function of (seed, tensor_id, step, j): Philox4x32 with 10 rounds, key =
// (seed low, seed high), counter = (j/4 low, j/4 high, tensor_id, step); the four output
// words give four normals by Box-Muller on the word pairs (x0,x1) and (x2,x3):
//   u1 = ((xa >> 8) + 1) * 2^-24 in (0,1],  u2 = (xb >> 8) * 2^-24 in [0,1)   (exact in fp32)
//   r = sqrt(-2 ln u1),  z = r cos(2 pi u2),  r sin(2 pi u2).
//
// Accuracy: an exhaustive scan over all 2^24 inputs of each factor (dp_debug_noise_error_scan,
// checked by a GPU test) gives max relative error 9.6e-8 for the fp32 radius and max absolute
// error 5.3e-8 for the fp32 cosine / sine; with the 2^-24 rounding of the product the error of
// z is at most r * 2.1e-7, i.e. below 1e-6 while r <= 4.5.  Pairs with a larger radius
// (4e-5 of them) take a float64 path, whose only error is the final rounding to fp32.
#pragma once

#include <stdint.h>

namespace dpg {

struct NoiseKey {
  uint32_t k0, k1;         // seed low / high word
  uint32_t tensor_id, step;
};

// The step word of a launch: the host's value plus, when a device counter is registered
// (dp_noise_step_device), the counter's current value -- so that a captured CUDA graph draws
// fresh noise at every replay.
__device__ __forceinline__ uint32_t effective_step(uint32_t step, const uint32_t* step_dev) {
  return step_dev ? step + __ldg(step_dev) : step;
}

struct U4 { uint32_t x, y, z, w; };

__device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                            uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // one 32x32->64 multiply per half round gives both product words
    const unsigned long long p0 = (unsigned long long)0xD2511F53u * c0;
    const unsigned long long p1 = (unsigned long long)0xCD9E8D57u * c2;
    const uint32_t hi0 = uint32_t(p0 >> 32), lo0 = uint32_t(p0);
    const uint32_t hi1 = uint32_t(p1 >> 32), lo1 = uint32_t(p1);
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return U4{c0, c1, c2, c3};
}

// float64 evaluation for the rare large radii; kept out of line so that the common path stays
// small in the instruction cache
static __device__ __noinline__ void box_muller_tail(uint32_t xa, uint32_t xb, float& za, float& zb) {
  const double r = sqrt(-2.0 * log(double((xa >> 8) + 1u) * 5.9604644775390625e-08));
  double s, c;
  sincospi(double(xb >> 8) * 1.1920928955078125e-07, &s, &c);
  za = float(r * c);
  zb = float(r * s);
}

// fp32 radius and direction of one pair; the same expressions are scanned exhaustively over
// all 2^24 inputs by dp_debug_noise_error_scan to bound their error.
__device__ __forceinline__ float bm_t_f32(uint32_t ka) {              // -2 ln u1
  return -2.0f * logf(float(ka + 1u) * 5.9604644775390625e-08f);      // u1 = (ka+1) * 2^-24
}
__device__ __forceinline__ void bm_dir_f32(uint32_t kb, float& s, float& c) {
  sincospif(float(kb) * 1.1920928955078125e-07f, &s, &c);             // 2 * u2, exact
}

// fp32 path while r^2 <= kTailT; see noise_kernel.cu for how the threshold follows from the
// measured error of the two factors
#ifndef DPG_NOISE_TAIL_T
#define DPG_NOISE_TAIL_T 20.25f
#endif

__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& za, float& zb) {
  const float t = bm_t_f32(xa >> 8);
  if (t <= DPG_NOISE_TAIL_T) {
    const float r = __fsqrt_rn(t);
    float s, c;
    bm_dir_f32(xb >> 8, s, c);
    za = r * c;
    zb = r * s;
  } else {
    box_muller_tail(xa, xb, za, zb);
  }
}

// the four normals of counter q (elements 4q .. 4q+3 of the tensor)
__device__ __forceinline__ void normals4(unsigned long long q, const NoiseKey& key, float (&z)[4]) {
  const U4 x = philox4x32_10(uint32_t(q), uint32_t(q >> 32), key.tensor_id, key.step, key.k0, key.k1);
  box_muller(x.x, x.y, z[0], z[1]);
  box_muller(x.z, x.w, z[2], z[3]);
}

// Eq. 3 on one element: scale * (v + amp * z)
__device__ __forceinline__ float noised(float v, float z, float amp, float scale) {
  return scale * fmaf(amp, z, v);
}

}  // namespace dpg
