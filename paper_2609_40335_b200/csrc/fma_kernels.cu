// fp32-FMA kernels for linear layers: the DP_F32 path (fp32 tensors need better than TF32
// accuracy) and the cross-check path for DP_BF16.  Any shape, no alignment rules.
//   ghost  : sq[i] += sum_{t,s} (a_t.a_s)(g_t.g_s)            (Eq. 4 - Eq. 5 over T tokens)
//   direct : sq[i] += sum_{r,c} (sum_t G[t,r] A[t,c])^2
//   clipped sum: out = beta*out + sum_i R_i G_i^T A_i          (inner sum of Eq. 3)
#include "dp_common.cuh"
#include "fma_kernels.cuh"

namespace dpg {

namespace {

template <typename T>
__global__ void ghost_norm_fma_kernel(const T* __restrict__ A, long long lda, int d,
                                      const T* __restrict__ G, long long ldg, int p, int Tn,
                                      float* __restrict__ sq) {
  __shared__ float red[32];
  const int i = blockIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const T* Ai = A + size_t(i) * Tn * lda;
  const T* Gi = G + size_t(i) * Tn * ldg;
  const long long npairs = (long long)Tn * (Tn + 1) / 2;
  float acc = 0.f;
  int t = 0, s = 0;                       // pair index -> (t, s), s >= t, walked incrementally
  long long cur = 0;
  for (long long pr = w; pr < npairs; pr += nw) {
    while (cur < pr) {                    // advance the (t, s) cursor to pair pr
      const long long left = Tn - s - 1;  // pairs left in row t after (t, s)
      const long long jump = pr - cur;
      if (jump <= left) { s += (int)jump; cur = pr; }
      else { cur += left + 1; ++t; s = t; }
    }
    float da = 0.f, dg = 0.f;
    for (int k = lane; k < d; k += 32) da = fmaf(to_f32(Ai[t * lda + k]), to_f32(Ai[s * lda + k]), da);
    for (int k = lane; k < p; k += 32) dg = fmaf(to_f32(Gi[t * ldg + k]), to_f32(Gi[s * ldg + k]), dg);
    da = warp_sum(da);
    dg = warp_sum(dg);
    acc += (t == s ? 1.f : 2.f) * da * dg;
  }
  const float tot = block_sum(lane == 0 ? acc : 0.f, red);
  if (threadIdx.x == 0) sq[i] += tot;
}

template <typename T>
__global__ void direct_norm_fma_kernel(const T* __restrict__ A, long long lda, int d,
                                       const T* __restrict__ G, long long ldg, int p, int Tn,
                                       float* __restrict__ sq) {
  __shared__ float red[32];
  const int i = blockIdx.x;
  const T* Ai = A + size_t(i) * Tn * lda;
  const T* Gi = G + size_t(i) * Tn * ldg;
  const long long n = (long long)d * p;
  float acc = 0.f;
  for (long long e = threadIdx.x; e < n; e += blockDim.x) {
    const int r = int(e / d), c = int(e - (long long)r * d);
    float v = 0.f;
    for (int t = 0; t < Tn; ++t) v = fmaf(to_f32(Gi[t * ldg + r]), to_f32(Ai[t * lda + c]), v);
    acc = fmaf(v, v, acc);
  }
  const float tot = block_sum(acc, red);
  if (threadIdx.x == 0) sq[i] += tot;
}

// 64 x 64 output tile per block of 256 threads, 16 token rows per shared-memory step
template <typename T>
__global__ void clip_accumulate_fma_kernel(const T* __restrict__ A, long long lda, int d,
                                           const T* __restrict__ G, long long ldg, int p, int B,
                                           int Tn, const float* __restrict__ clip,
                                           float* __restrict__ out, long long ldo, float beta) {
  __shared__ float Gs[16][64 + 1];
  __shared__ float As[16][64 + 1];
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  const long long K = (long long)B * Tn;
  for (long long k0 = 0; k0 < K; k0 += 16) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      const int kk = e >> 6, c = e & 63;
      const long long k = k0 + kk;
      float g = 0.f, a = 0.f;
      if (k < K) {
        const float r = clip[k / Tn];
        if (m0 + c < p) g = r * to_f32(G[k * ldg + m0 + c]);
        if (n0 + c < d) a = to_f32(A[k * lda + n0 + c]);
      }
      Gs[kk][c] = g;
      As[kk][c] = a;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float gv[4], av[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) { gv[j] = Gs[kk][ty * 4 + j]; av[j] = As[kk][tx * 4 + j]; }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(gv[a], av[b], acc[a][b]);
    }
    __syncthreads();
  }
  for (int a = 0; a < 4; ++a)
    for (int b = 0; b < 4; ++b) {
      const int r = m0 + ty * 4 + a, c = n0 + tx * 4 + b;
      if (r < p && c < d) {
        float* o = out + size_t(r) * ldo + c;
        *o = (beta != 0.f) ? (*o + acc[a][b]) : acc[a][b];
      }
    }
}

// <g_in_i, g_out_i> = sum_{t,s} G_lm[i,s,id_t] * (g_emb_t . a_lm_s)   (expansion of Eq. 11's
// inner product); one block per (example, 16-token slab of t), one warp per (t, s) pair.
template <typename T>
__global__ void cross_term_fma_kernel(const int* __restrict__ ids, const T* __restrict__ Ge,
                                      long long ldge, const T* __restrict__ Al, long long ldal,
                                      const T* __restrict__ Gl, long long ldgl, int Tn, int d, int V,
                                      int slabs, float* __restrict__ partials,
                                      int* __restrict__ dev_status) {
  __shared__ float red[32];
  const int i = blockIdx.x / slabs, slab = blockIdx.x % slabs;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int t_lo = slab * 16, t_hi = min(Tn, t_lo + 16);
  float acc = 0.f;
  for (int t = t_lo; t < t_hi; ++t) {
    const int id = ids[size_t(i) * Tn + t];
    if (id < 0 || id >= V) {
      if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, DP_DEV_BAD_ID);
      continue;
    }
    const T* g = Ge + (size_t(i) * Tn + t) * ldge;
    for (int s = w; s < Tn; s += nw) {
      const T* a = Al + (size_t(i) * Tn + s) * ldal;
      float dot = 0.f;
      for (int k = lane; k < d; k += 32) dot = fmaf(to_f32(g[k]), to_f32(a[k]), dot);
      dot = warp_sum(dot);
      acc = fmaf(to_f32(Gl[(size_t(i) * Tn + s) * ldgl + id]), dot, acc);
    }
  }
  const float tot = block_sum(lane == 0 ? acc : 0.f, red);
  if (threadIdx.x == 0) partials[blockIdx.x] = tot;
}

__global__ void clip_factors_kernel(const float* __restrict__ sq, int B, float C,
                                    float* __restrict__ clip, float* __restrict__ norms,
                                    const float* __restrict__ extra, float* __restrict__ sq_out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B) return;
  float s = sq[i];
  if (extra) {                 // a second accumulator of squared norms joins first (fixed order)
    s += extra[i];
    sq_out[i] = s;
  }
  if (clip) clip[i] = clip_from_sq(s, C);
  if (norms) norms[i] = __fsqrt_rn(s);
}

}  // namespace

template <typename T>
static dp_status norms_fma_t(const dp_linear_desc& L, int mode, int B, int Tn, float* sq,
                             cudaStream_t st) {
  if (mode == DP_NORM_GHOST)
    ghost_norm_fma_kernel<T><<<B, 256, 0, st>>>((const T*)L.A, L.lda, L.d, (const T*)L.G, L.ldg,
                                               L.p, Tn, sq);
  else
    direct_norm_fma_kernel<T><<<B, 256, 0, st>>>((const T*)L.A, L.lda, L.d, (const T*)L.G, L.ldg,
                                                L.p, Tn, sq);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_norms_fma(const dp_linear_desc& L, dp_dtype dt, int mode, int B, int T, float* sq,
                           cudaStream_t st) {
  return dt == DP_F32 ? norms_fma_t<float>(L, mode, B, T, sq, st)
                      : norms_fma_t<__nv_bfloat16>(L, mode, B, T, sq, st);
}

dp_status launch_clip_accumulate_fma(const void* A, int64_t lda, const void* G, int64_t ldg,
                                     dp_dtype dt, int B, int T, int d, int p, const float* clip,
                                     float* out, int64_t ldo, float beta, cudaStream_t st) {
  dim3 grid(ceil_div(d, 64), ceil_div(p, 64));
  if (dt == DP_F32)
    clip_accumulate_fma_kernel<float><<<grid, 256, 0, st>>>((const float*)A, lda, d, (const float*)G,
                                                           ldg, p, B, T, clip, out, ldo, beta);
  else
    clip_accumulate_fma_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
        (const __nv_bfloat16*)A, lda, d, (const __nv_bfloat16*)G, ldg, p, B, T, clip, out, ldo, beta);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_cross_term_fma(const int* ids, const void* Ge, int64_t ldge, const void* Al,
                                int64_t ldal, const void* Gl, int64_t ldgl, dp_dtype dt, int B,
                                int T, int d, int V, float* partials, int* dev_status,
                                cudaStream_t st) {
  const int slabs = ceil_div(T, 16);
  if (dt == DP_F32)
    cross_term_fma_kernel<float><<<B * slabs, 256, 0, st>>>(ids, (const float*)Ge, ldge,
                                                          (const float*)Al, ldal, (const float*)Gl,
                                                          ldgl, T, d, V, slabs, partials, dev_status);
  else
    cross_term_fma_kernel<__nv_bfloat16><<<B * slabs, 256, 0, st>>>(
        ids, (const __nv_bfloat16*)Ge, ldge, (const __nv_bfloat16*)Al, ldal,
        (const __nv_bfloat16*)Gl, ldgl, T, d, V, slabs, partials, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_clip_factors(const float* sq, int B, float C, float* clip, float* norms,
                              cudaStream_t st, const float* extra, float* sq_out) {
  clip_factors_kernel<<<ceil_div(B, 128), 128, 0, st>>>(sq, B, C, clip, norms, extra, sq_out);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
