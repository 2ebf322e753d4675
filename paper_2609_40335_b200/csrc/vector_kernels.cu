// Parameters that act element-wise along the feature axis: biases and LayerNorm gains / shifts.
//
// A bias b in z = W a + b sees the back-propagated signal of every token (Eq. 4 with a constant
// input 1), so its per-example gradient is v_i = sum_t G[i,t,:]; a LayerNorm gain sees
// v_i = sum_t G[i,t,:] * X[i,t,:] with X the normalised input and G the gradient at the
// LayerNorm output (its shift is a bias).  These kernels give
//     norms:        sq[i] += || v_i ||^2                                   (one more block of Eq. 6)
//     clipped sum:  out = beta*out + sum_i R_i v_i  [+ Gaussian noise]      (Eq. 3)
// Both are single streaming passes over G (and X): HBM-bound, 2*T*p (or 4*T*p) bytes per example.
// Summation orders are fixed (warp w takes rows w, w+8, ...; partial sums are combined in
// warp / split order), so results are deterministic.
#include <algorithm>
#include <cstring>

#include "dp_common.cuh"
#include "noise_device.cuh"
#include "vector_kernels.cuh"

namespace dpg {

namespace {

constexpr int kVecCols = 256;        // columns per block (8 per lane)
// 16-byte row loads in flight per lane: eight G rows for a bias, four G and four X rows for a
// LayerNorm gain (kept unconverted: 32 registers), so that four 256-thread blocks
// (<= 64 registers per thread) fit on an SM
constexpr int kVecBatchBias = 8;
constexpr int kVecBatchGain = 4;

struct VecParam {
  const void* G;
  const void* X;          // multiplier or nullptr
  long long ldg, ldx;
  float* out;             // clipped-sum destination (p floats)
  int p;
  int slab_begin;         // first 256-column slab of this parameter in the launch
  int col_begin;          // first column of this parameter in the concatenated partial rows
  uint32_t tensor_id;
};

struct VecParams {
  VecParam prm[kVecMaxParams];
  int n, B, T;
  int total_slabs, total_cols;
};

__device__ __forceinline__ int find_param(const VecParams& P, int slab) {
  int k = 0;
  while (k + 1 < P.n && slab >= P.prm[k + 1].slab_begin) ++k;
  return k;
}

// Eight consecutive columns of one row, kept as loaded (a bf16 row chunk stays one 16-byte
// register quad until it is consumed, so twice as many loads fit in flight per thread).
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p, int nvalid, bool vec) {
    if (vec && nvalid >= 8) {
      q = *reinterpret_cast<const uint4*>(p);
    } else {
      uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (e < nvalid) w[e >> 1] |= uint32_t(__bfloat16_as_ushort(p[e])) << (16 * (e & 1));
      q = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      v[2 * e] = __uint_as_float(w[e] << 16);
      v[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
  }
};
template <> struct Raw8<float> {
  float v8[8];
  __device__ __forceinline__ void load(const float* p, int nvalid, bool vec) { load8<float>(p, nvalid, vec, v8); }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = v8[e];
  }
};

// sum over the rows [r0, r1) (stride 8 from warp w) of weight(row) * G[row, cols] * X[row, cols].
// All loads of a batch are issued before any is consumed; rows past r1 re-read row r1-1 with
// weight 0, so the loads are unconditional.  The example of a row (for its clip factor) is
// tracked by stepping, not by a division per row.
template <typename T, bool kWeighted, bool kHasX>
__device__ __forceinline__ void stream_rows_t(const VecParam& q, long long row_base, int r0, int r1,
                                              int c, int nvalid, int Tn, const float* clip,
                                              float (&acc)[8]) {
  // fp32 chunks are twice as large in registers: half the batch
  constexpr int kBatch = (kHasX ? kVecBatchGain : kVecBatchBias) / (sizeof(T) == 2 ? 1 : 2);
  const int w = threadIdx.x >> 5;
  if (r0 + w >= r1) return;
  const T* G = static_cast<const T*>(q.G) + row_base * q.ldg + c;
  const T* X = kHasX ? static_cast<const T*>(q.X) + row_base * q.ldx + c : nullptr;
  const bool gvec = ((reinterpret_cast<uintptr_t>(q.G) & 15) == 0) && ((q.ldg * sizeof(T)) % 16 == 0);
  const bool xvec = kHasX && ((reinterpret_cast<uintptr_t>(q.X) & 15) == 0) && ((q.ldx * sizeof(T)) % 16 == 0);
  // example and token of the first row this warp takes
  long long ex = kWeighted ? (row_base + r0 + w) / Tn : 0;
  int t = kWeighted ? int((row_base + r0 + w) - ex * Tn) : 0;
  for (int rr = r0 + w; rr < r1; rr += 8 * kBatch) {
    Raw8<T> g[kBatch], x[kHasX ? kBatch : 1];
    float wt[kBatch];
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int r = rr + 8 * b;
      const int rc = min(r, r1 - 1);
      g[b].load(G + size_t(rc) * q.ldg, nvalid, gvec);
      if (kHasX) x[kHasX ? b : 0].load(X + size_t(rc) * q.ldx, nvalid, xvec);
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      float f = 1.f;
      if (kWeighted) {
        long long eb = ex;
        int tb = t + 8 * b;
        while (tb >= Tn) { tb -= Tn; ++eb; }
        f = (rr + 8 * b < r1) ? __ldg(clip + eb) : 0.f;      // eb < B whenever the row exists
      }
      wt[b] = (rr + 8 * b < r1) ? f : 0.f;
    }
    if (kWeighted) {
      t += 8 * kBatch;
      while (t >= Tn) { t -= Tn; ++ex; }
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      float gv[8], xv[8];
      g[b].unpack(gv);
      if (kHasX) x[kHasX ? b : 0].unpack(xv);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float v = kHasX ? gv[e] * xv[e] : gv[e];
        acc[e] = fmaf(wt[b], v, acc[e]);
      }
    }
  }
}

template <typename T, bool kWeighted>
__device__ __forceinline__ void stream_rows(const VecParam& q, long long row_base, int r0, int r1,
                                            int c, int nvalid, int Tn, const float* clip,
                                            float (&acc)[8]) {
  if (q.X) stream_rows_t<T, kWeighted, true>(q, row_base, r0, r1, c, nvalid, Tn, clip, acc);
  else stream_rows_t<T, kWeighted, false>(q, row_base, r0, r1, c, nvalid, Tn, clip, acc);
}

// grid = (slabs of all parameters, examples): || sum_t G*X ||^2 restricted to the block's columns
template <typename T>
__global__ void __launch_bounds__(256, 4)
vector_norm_kernel(const __grid_constant__ VecParams P, float* __restrict__ partials, int n_per,
                   int col0_partial) {
  __shared__ float part[8][kVecCols];
  __shared__ float red[32];
  const int slab = blockIdx.x, i = blockIdx.y;
  const VecParam& q = P.prm[find_param(P, slab)];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = (slab - q.slab_begin) * kVecCols + lane * 8;
  const int nvalid = min(8, q.p - c);
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  if (nvalid > 0) stream_rows<T, false>(q, (long long)i * P.T, 0, P.T, c, nvalid, P.T, nullptr, acc);
#pragma unroll
  for (int e = 0; e < 8; ++e) part[w][lane * 8 + e] = acc[e];
  __syncthreads();
  float v = 0.f;
#pragma unroll
  for (int ww = 0; ww < 8; ++ww) v += part[ww][threadIdx.x];
  const float s = block_sum(v * v, red);
  if (threadIdx.x == 0) partials[size_t(i) * n_per + col0_partial + slab] = s;
}

// grid = (slabs of all parameters, row splits): partial clipped sums of the block's columns
template <typename T>
__global__ void __launch_bounds__(256, 4)
vector_sum_kernel(const __grid_constant__ VecParams P, const float* __restrict__ clip,
                  int rows_per_split, float* __restrict__ partial) {
  __shared__ float part[8][kVecCols];
  const int slab = blockIdx.x, split = blockIdx.y;
  const VecParam& q = P.prm[find_param(P, slab)];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = (slab - q.slab_begin) * kVecCols + lane * 8;
  const int nvalid = min(8, q.p - c);
  const long long rows = (long long)P.B * P.T;
  const long long r0 = (long long)split * rows_per_split;
  const int nrows = (int)max(0LL, min((long long)rows_per_split, rows - r0));
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  if (nvalid > 0) stream_rows<T, true>(q, r0, 0, nrows, c, nvalid, P.T, clip, acc);
#pragma unroll
  for (int e = 0; e < 8; ++e) part[w][lane * 8 + e] = acc[e];
  __syncthreads();
  const int cc = (slab - q.slab_begin) * kVecCols + threadIdx.x;
  if (cc < q.p) {
    float v = 0.f;
#pragma unroll
    for (int ww = 0; ww < 8; ++ww) v += part[ww][threadIdx.x];
    partial[size_t(split) * P.total_cols + q.col_begin + cc] = v;
  }
}

// out = beta*out + sum over row splits (in split order), then the Gaussian mechanism of Eq. 3
__global__ void __launch_bounds__(256)
vector_combine_kernel(const __grid_constant__ VecParams P, const float* __restrict__ partial,
                      int nsplit, float beta, int with_noise, float amp, float scale, uint32_t k0,
                      uint32_t k1, uint32_t step, const uint32_t* __restrict__ step_dev) {
  const int slab = blockIdx.x;
  const VecParam& q = P.prm[find_param(P, slab)];
  const int cc = (slab - q.slab_begin) * kVecCols + threadIdx.x;
  if (cc >= q.p) return;
  float v = 0.f;
  for (int s = 0; s < nsplit; ++s) v += partial[size_t(s) * P.total_cols + q.col_begin + cc];
  if (beta != 0.f) v += q.out[cc];
  if (with_noise) {
    const NoiseKey key{k0, k1, q.tensor_id, effective_step(step, step_dev)};
    float z[4];
    normals4((unsigned long long)(cc >> 2), key, z);
    const int e = cc & 3;
    v = noised(v, e == 0 ? z[0] : e == 1 ? z[1] : e == 2 ? z[2] : z[3], amp, scale);
  }
  q.out[cc] = v;
}

}  // namespace

namespace {

int fill_params(VecParams& P, const dp_vector_desc* prm, int n0, int n1, float* const* outs,
                const uint32_t* tensor_ids, int B, int T) {
  memset(&P, 0, sizeof(P));
  int slabs = 0, cols = 0;
  for (int k = n0; k < n1; ++k) {
    VecParam& q = P.prm[k - n0];
    q.G = prm[k].G; q.X = prm[k].X; q.ldg = prm[k].ldg; q.ldx = prm[k].ldx; q.p = prm[k].p;
    q.out = outs ? outs[k] : nullptr;
    q.tensor_id = tensor_ids ? tensor_ids[k] : 0u;
    q.slab_begin = slabs; q.col_begin = cols;
    slabs += ceil_div(prm[k].p, kVecCols);
    cols += prm[k].p;
  }
  P.n = n1 - n0; P.B = B; P.T = T; P.total_slabs = slabs; P.total_cols = cols;
  return slabs;
}

}  // namespace

int vector_total_slabs(const dp_vector_desc* prm, int n) {
  int s = 0;
  for (int k = 0; k < n; ++k) s += ceil_div(prm[k].p, kVecCols);
  return s;
}

// row splits of the clipped-sum pass: enough blocks for about eight per SM, >= 64 rows each
int vector_row_splits(const dp_vector_desc* prm, int n, int B, int T, int sms) {
  const long long rows = (long long)B * T;
  const int slabs = std::max(1, vector_total_slabs(prm, std::min(n, kVecMaxParams)));
  long long ns = std::max<long long>(1, (8LL * sms) / slabs);
  ns = std::min<long long>(ns, std::max<long long>(1, rows / 64));
  return (int)ns;
}

dp_status launch_vector_norms(const dp_vector_desc* prm, int n, dp_dtype dt, int B, int T,
                              float* partials, int n_per, cudaStream_t st) {
  int col0 = 0;
  for (int n0 = 0; n0 < n; n0 += kVecMaxParams) {
    const int n1 = std::min(n, n0 + kVecMaxParams);
    VecParams P;
    const int slabs = fill_params(P, prm, n0, n1, nullptr, nullptr, B, T);
    dim3 grid(slabs, B);
    if (dt == DP_F32) vector_norm_kernel<float><<<grid, 256, 0, st>>>(P, partials, n_per, col0);
    else vector_norm_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(P, partials, n_per, col0);
    DP_LAUNCH_OK();
    col0 += slabs;
  }
  return DP_OK;
}

dp_status launch_vector_sums(const dp_vector_desc* prm, int n, dp_dtype dt, int B, int T,
                             const float* clip, float* const* outs, float beta, int with_noise,
                             float amp, float scale, uint64_t seed, const uint32_t* tensor_ids,
                             uint32_t step, float* partial_ws, cudaStream_t st) {
  const int sms = sm_count();
  const long long rows = (long long)B * T;
  for (int n0 = 0; n0 < n; n0 += kVecMaxParams) {
    const int n1 = std::min(n, n0 + kVecMaxParams);
    VecParams P;
    const int slabs = fill_params(P, prm, n0, n1, outs, tensor_ids, B, T);
    int nsplit = vector_row_splits(prm + n0, n1 - n0, B, T, sms);
    const int rps = (int)((rows + nsplit - 1) / nsplit);
    nsplit = (int)((rows + rps - 1) / rps);
    dim3 grid(slabs, nsplit);
    if (dt == DP_F32) vector_sum_kernel<float><<<grid, 256, 0, st>>>(P, clip, rps, partial_ws);
    else vector_sum_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(P, clip, rps, partial_ws);
    DP_LAUNCH_OK();
    vector_combine_kernel<<<slabs, 256, 0, st>>>(P, partial_ws, nsplit, beta, with_noise, amp, scale,
                                                uint32_t(seed), uint32_t(seed >> 32), step, g_step_dev);
    DP_LAUNCH_OK();
  }
  return DP_OK;
}

}  // namespace dpg
