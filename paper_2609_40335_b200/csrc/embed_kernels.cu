// Embedding-table kernels: per-example ghost norm by token-id equality, stable counting sort
// of token positions, and the clipped segmented row sum (scatter-add without atomics).
//
// An embedding is a linear layer whose input is the one-hot row of the token, so Eq. 4 gives
// e_{id_t} g_t^T per token and the per-example gradient has one row per DISTINCT token:
//   || g_i ||_F^2 = sum over distinct v of || sum_{t: id_t = v} g_t ||^2
//                 = sum_{t,s} [id_t == id_s] (g_t . g_s).
#include "dp_common.cuh"
#include "fma_kernels.cuh"

namespace dpg {

namespace {

// ------------------------------------------------------------------ norm kernel
// One block per (example, 256-column slab).  Tokens are grouped by their first occurrence
// (warp-level id matching, then a scan over earlier tokens for group leaders), ordered by
// (first occurrence, position), and every thread walks the ordered rows for its two columns:
// each row of G is read exactly once.
template <typename T>
__global__ void __launch_bounds__(128)
embed_norm_kernel(const int* __restrict__ ids, const T* __restrict__ G, long long ldg, int Tn, int d,
                  int V, int slabs, float* __restrict__ partials, int* __restrict__ first_occ,
                  int* __restrict__ dev_status) {
  extern __shared__ int sm_i[];
  int* s_id = sm_i;              // token id, -1 if out of range
  int* s_fo = sm_i + Tn;         // first occurrence
  int* s_ord = sm_i + 2 * Tn;    // rows ordered by (first occurrence, position); sign bit = group end
  __shared__ float red[32];
  const int i = blockIdx.x / slabs, slab = blockIdx.x % slabs;
  const int lane = threadIdx.x & 31;

  for (int t = threadIdx.x; t < Tn; t += blockDim.x) {
    int id = ids[size_t(i) * Tn + t];
    if (id < 0 || id >= V) {
      id = -1;
      if (dev_status) atomicOr(dev_status, DP_DEV_BAD_ID);
    }
    s_id[t] = id;
  }
  __syncthreads();

  // first occurrence: match inside the warp's 32-token window, leaders scan earlier windows
  const int t_round = (Tn + 31) & ~31;
  for (int t = threadIdx.x; t < t_round; t += blockDim.x) {
    const bool live = t < Tn;
    const int id = live ? s_id[t] : -2 - lane;             // unique sentinel for padding lanes
    const int key = (id == -1) ? -2 - 64 - lane : id;      // bad ids never match anything
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    const int leader = __ffs(peers) - 1;
    const int base = t - lane;
    int fo = base + leader;
    if (lane == leader && live && id >= 0) {
      for (int s = 0; s < base; ++s)
        if (s_id[s] == id) { fo = s; break; }
    }
    fo = __shfl_sync(0xffffffffu, fo, leader);
    if (live) s_fo[t] = (id >= 0) ? fo : t;
  }
  __syncthreads();

  // rank of token t in the order (first occurrence, position)
  for (int t = threadIdx.x; t < Tn; t += blockDim.x) {
    const int fo = s_fo[t];
    int rank = 0;
    for (int s = 0; s < Tn; ++s) {
      const int f = s_fo[s];
      rank += (f < fo) || (f == fo && s < t);
    }
    s_ord[rank] = t;
    if (slab == 0 && first_occ) first_occ[size_t(i) * Tn + t] = fo;
  }
  __syncthreads();
  // mark the last row of every group in the top bit (two passes: read all, then write)
  unsigned end_mask = 0;                   // bit k: row r = threadIdx.x + k*blockDim.x ends a group
  for (int r = threadIdx.x, k = 0; r < Tn; r += blockDim.x, ++k) {
    const bool end = (r == Tn - 1) || (s_fo[s_ord[r + 1]] != s_fo[s_ord[r]]);
    end_mask |= (end ? 1u : 0u) << k;
  }
  __syncthreads();
  for (int r = threadIdx.x, k = 0; r < Tn; r += blockDim.x, ++k)
    if ((end_mask >> k) & 1u) s_ord[r] |= int(0x80000000u);
  __syncthreads();

  // grouped row sums for this thread's two columns
  const int c = slab * kEmbedColsPerBlock + 2 * threadIdx.x;
  float tot = 0.f;
  if (c < d) {
    const bool two = (c + 1 < d);
    const T* Gi = G + size_t(i) * Tn * ldg + c;
    float r0 = 0.f, r1 = 0.f;
#pragma unroll 4
    for (int r = 0; r < Tn; ++r) {
      const int o = s_ord[r];
      const int t = o & 0x7fffffff;
      if (s_id[t] >= 0) {
        r0 += to_f32(Gi[size_t(t) * ldg]);
        if (two) r1 += to_f32(Gi[size_t(t) * ldg + 1]);
      }
      if (o < 0) {
        tot = fmaf(r0, r0, tot);
        tot = fmaf(r1, r1, tot);
        r0 = 0.f; r1 = 0.f;
      }
    }
  }
  const float s = block_sum(tot, red);
  if (threadIdx.x == 0) partials[size_t(i) * slabs + slab] = s;
}

// ------------------------------------------------------------------ sort kernels
__global__ void sort_hist_kernel(const int* __restrict__ ids, int n, int V, int* __restrict__ counts,
                                 int* __restrict__ dev_status) {
  const int chunk = blockIdx.x;
  const int j = chunk * kSortChunk + threadIdx.x;
  if (j >= n) return;
  const int id = ids[j];
  if (id < 0 || id >= V) {
    if (dev_status) atomicOr(dev_status, DP_DEV_BAD_ID);
    return;
  }
  atomicAdd(&counts[size_t(chunk) * V + id], 1);
}

// counts[c][v] -> number of id v in chunks before c; seg[v] = total count of v
__global__ void sort_chunk_prefix_kernel(int* __restrict__ counts, int chunks, int V,
                                         int* __restrict__ seg) {
  const int v = blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= V) return;
  int run = 0;
  for (int c = 0; c < chunks; ++c) {
    const int x = counts[size_t(c) * V + v];
    counts[size_t(c) * V + v] = run;
    run += x;
  }
  seg[v] = run;
}

// in-place exclusive scan of seg[0..V] (seg[V] receives the total); single block
__global__ void __launch_bounds__(1024) sort_scan_kernel(int* __restrict__ seg, int V) {
  __shared__ int part[1024];
  const int per = (V + 1 + 1023) / 1024;
  const int lo = threadIdx.x * per, hi = min(V + 1, lo + per);
  int s = 0;
  for (int v = lo; v < hi; ++v) s += (v < V) ? seg[v] : 0;
  part[threadIdx.x] = s;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {       // Hillis-Steele inclusive scan
    const int x = (threadIdx.x >= off) ? part[threadIdx.x - off] : 0;
    __syncthreads();
    part[threadIdx.x] += x;
    __syncthreads();
  }
  int run = part[threadIdx.x] - s;
  for (int v = lo; v < hi; ++v) {
    const int x = (v < V) ? seg[v] : 0;
    seg[v] = run;
    run += x;
  }
}

__global__ void __launch_bounds__(kSortChunk)
sort_place_kernel(const int* __restrict__ ids, int n, int V, const int* __restrict__ counts,
                  const int* __restrict__ seg, int* __restrict__ perm) {
  __shared__ int s_id[kSortChunk];
  const int chunk = blockIdx.x;
  const int j = chunk * kSortChunk + threadIdx.x;
  int id = (j < n) ? ids[j] : -1;
  if (id < 0 || id >= V) id = -1;
  s_id[threadIdx.x] = id;
  __syncthreads();
  if (id < 0) return;
  int r = 0;
  for (int s = 0; s < (int)threadIdx.x; ++s) r += (s_id[s] == id);
  perm[seg[id] + counts[size_t(chunk) * V + id] + r] = j;
}

// ------------------------------------------------------------------ segmented row sum
// grid = (sorted positions, 128-column slices); only the block sitting on the first sorted
// position of a token id works.  8 warps take rows k = w, w+8, ... of the segment in order and
// their partial sums are combined in warp order, so the result does not depend on timing.
template <typename T>
__global__ void __launch_bounds__(256)
embed_scatter_kernel(const int* __restrict__ ids, const T* __restrict__ G, long long ldg, int Tn,
                     int d, const float* __restrict__ clip, const int* __restrict__ perm,
                     const int* __restrict__ seg, int V, float* __restrict__ out, long long ldo,
                     float beta) {
  __shared__ float part[8][128];
  const int k0 = blockIdx.x;
  if (k0 >= seg[V]) return;
  const int pos0 = perm[k0];
  const int v = ids[pos0];
  if (seg[v] != k0) return;                    // not the head of its segment
  const int n = seg[v + 1] - k0;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int c = blockIdx.y * 128 + lane * 4;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  if (c < d) {
#pragma unroll 4
    for (int k = w; k < n; k += 8) {
      const int pos = perm[k0 + k];
      const float r = clip[pos / Tn];
      const T* g = G + size_t(pos) * ldg + c;
      a0 = fmaf(r, to_f32(g[0]), a0);
      if (c + 1 < d) a1 = fmaf(r, to_f32(g[1]), a1);
      if (c + 2 < d) a2 = fmaf(r, to_f32(g[2]), a2);
      if (c + 3 < d) a3 = fmaf(r, to_f32(g[3]), a3);
    }
  }
  part[w][lane * 4 + 0] = a0; part[w][lane * 4 + 1] = a1;
  part[w][lane * 4 + 2] = a2; part[w][lane * 4 + 3] = a3;
  __syncthreads();
  if (threadIdx.x < 128) {
    const int cc = blockIdx.y * 128 + threadIdx.x;
    if (cc < d) {
      float s = 0.f;
#pragma unroll
      for (int ww = 0; ww < 8; ++ww) s += part[ww][threadIdx.x];
      float* o = out + size_t(v) * ldo + cc;
      *o = (beta != 0.f) ? (*o + s) : s;
    }
  }
}

}  // namespace

dp_status launch_embed_norms(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int B, int T,
                             int d, int V, float* partials, int* first_occ, int* dev_status,
                             cudaStream_t st) {
  const int slabs = ceil_div(d, kEmbedColsPerBlock);
  const size_t smem = size_t(3) * T * sizeof(int);
  static bool attr = false;
  if (!attr) {
    DP_CUDA_OK(cudaFuncSetAttribute(embed_norm_kernel<float>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    3 * kEmbedMaxT * (int)sizeof(int)));
    DP_CUDA_OK(cudaFuncSetAttribute(embed_norm_kernel<__nv_bfloat16>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    3 * kEmbedMaxT * (int)sizeof(int)));
    attr = true;
  }
  if (dt == DP_F32)
    embed_norm_kernel<float><<<B * slabs, 128, smem, st>>>(ids, (const float*)G, ldg, T, d, V, slabs,
                                                          partials, first_occ, dev_status);
  else
    embed_norm_kernel<__nv_bfloat16><<<B * slabs, 128, smem, st>>>(
        ids, (const __nv_bfloat16*)G, ldg, T, d, V, slabs, partials, first_occ, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_embed_sort(const int* ids, int n, int V, const EmbedSortWs& ws, int* dev_status,
                            cudaStream_t st) {
  DP_CUDA_OK(cudaMemsetAsync(ws.counts, 0, size_t(ws.chunks) * V * sizeof(int), st));
  sort_hist_kernel<<<ws.chunks, kSortChunk, 0, st>>>(ids, n, V, ws.counts, dev_status);
  DP_LAUNCH_OK();
  sort_chunk_prefix_kernel<<<ceil_div(V, 256), 256, 0, st>>>(ws.counts, ws.chunks, V, ws.seg);
  DP_LAUNCH_OK();
  sort_scan_kernel<<<1, 1024, 0, st>>>(ws.seg, V);
  DP_LAUNCH_OK();
  sort_place_kernel<<<ws.chunks, kSortChunk, 0, st>>>(ids, n, V, ws.counts, ws.seg, ws.perm);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_embed_scatter(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int n,
                               int T, int d, int V, const float* clip, const int* perm,
                               const int* seg, float* out, int64_t ldo, float beta,
                               cudaStream_t st) {
  // beta == 0: clear the table once, then every touched row is written as 0 + sum
  if (beta == 0.f) {
    DP_CUDA_OK(cudaMemset2DAsync(out, size_t(ldo) * sizeof(float), 0, size_t(d) * sizeof(float),
                                 size_t(V), st));
  }
  dim3 grid(n, ceil_div(d, 128));
  if (dt == DP_F32)
    embed_scatter_kernel<float><<<grid, 256, 0, st>>>(ids, (const float*)G, ldg, T, d, clip, perm,
                                                     seg, V, out, ldo, 1.f);
  else
    embed_scatter_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(ids, (const __nv_bfloat16*)G, ldg, T,
                                                             d, clip, perm, seg, V, out, ldo, 1.f);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
