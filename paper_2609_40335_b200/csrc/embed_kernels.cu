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

// ------------------------------------------------------------------ norm kernel
// One block (8 warps) per (example, 256-column slab).  Tokens are grouped by their first
// occurrence (warp-level id matching, then a scan over earlier tokens for group leaders) and
// ordered by (first occurrence, position).  The ordered rows are cut into 8 contiguous ranges
// at group boundaries, one per warp; a lane owns 8 columns, loads 8 rows at a time (16-byte
// loads, all in flight together) and folds them into running group sums.  Each row of G is
// read exactly once.
constexpr int kEmbedNormThreads = 256;
constexpr int kEmbedBatch = 8;

template <typename T>
__global__ void __launch_bounds__(kEmbedNormThreads)
embed_norm_kernel(const int* __restrict__ ids, const T* __restrict__ G, long long ldg, int Tn, int d,
                  int V, int slabs, float* __restrict__ partials, int* __restrict__ first_occ,
                  int* __restrict__ dev_status) {
  extern __shared__ int sm_i[];
  int* s_id = sm_i;              // token id, -1 if out of range
  int* s_fo = sm_i + Tn;         // first occurrence
  int* s_ord = sm_i + 2 * Tn;    // rows ordered by (first occurrence, position); sign bit = group end
  __shared__ float red[32];
  const int i = blockIdx.x / slabs, slab = blockIdx.x % slabs;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kEmbedNormThreads / 32;

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

  // this warp's range of ordered rows, snapped forward to group starts
  auto snap = [&](int r) {
    while (r > 0 && r < Tn && s_ord[r - 1] >= 0) ++r;      // previous row does not end a group
    return min(r, Tn);
  };
  const int per = (Tn + kWarps - 1) / kWarps;
  const int lo = snap(min(warp * per, Tn)), hi = snap(min((warp + 1) * per, Tn));

  const int c = slab * kEmbedColsPerBlock + 8 * lane;
  const int nvalid = min(8, d - c);
  float tot = 0.f;
  if (nvalid > 0) {
    const bool vec = ((reinterpret_cast<uintptr_t>(G) & 15) == 0) && ((ldg * sizeof(T)) % 16 == 0);
    const T* Gi = G + size_t(i) * Tn * ldg + c;
    float run[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) run[e] = 0.f;
    for (int r0 = lo; r0 < hi; r0 += kEmbedBatch) {
      float v[kEmbedBatch][8];
      int o[kEmbedBatch];
#pragma unroll
      for (int b = 0; b < kEmbedBatch; ++b) {
        const int r = r0 + b;
        o[b] = r < hi ? s_ord[r] : 0;
        const int t = o[b] & 0x7fffffff;
        if (r < hi && s_id[t] >= 0) {
          load8<T>(Gi + size_t(t) * ldg, nvalid, vec, v[b]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) v[b][e] = 0.f;
        }
      }
#pragma unroll
      for (int b = 0; b < kEmbedBatch; ++b) {
        if (r0 + b < hi) {
#pragma unroll
          for (int e = 0; e < 8; ++e) run[e] += v[b][e];
          if (o[b] < 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) { tot = fmaf(run[e], run[e], tot); run[e] = 0.f; }
          }
        }
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

// counts[c][v] -> number of id v in chunks before c; seg[v] = total count of v; block totals of
// seg (1024 ids per block) go to blk[] for the scan that follows
__global__ void __launch_bounds__(1024)
sort_chunk_prefix_kernel(int* __restrict__ counts, int chunks, int V, int* __restrict__ seg,
                         int* __restrict__ blk) {
  __shared__ int wsum[32];
  const int v = blockIdx.x * 1024 + threadIdx.x;
  int run = 0;
  if (v < V) {
    for (int c = 0; c < chunks; ++c) {
      const int x = counts[size_t(c) * V + v];
      counts[size_t(c) * V + v] = run;
      run += x;
    }
    seg[v] = run;
  }
  int s = run;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x < 32) {
    int t = wsum[threadIdx.x];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) blk[blockIdx.x] = t;
  }
}

// in-place exclusive scan of seg[0..V) (seg[V] receives the total): block b adds the totals of
// the blocks before it to a block-local scan of its 1024 entries
__global__ void __launch_bounds__(1024)
sort_scan_kernel(int* __restrict__ seg, int V, const int* __restrict__ blk) {
  __shared__ int wsum[32];
  __shared__ int base_s;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (w == 0) {
    int b = 0;
    for (int k = lane; k < (int)blockIdx.x; k += 32) b += blk[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b += __shfl_xor_sync(0xffffffffu, b, o);
    if (lane == 0) base_s = b;
  }
  const int v = blockIdx.x * 1024 + threadIdx.x;
  const int x = v < V ? seg[v] : 0;
  int inc = x;                                         // inclusive scan inside the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  if (lane == 31) wsum[w] = inc;
  __syncthreads();
  if (w == 0) {
    int t = wsum[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, t, o);
      if (lane >= o) t += y;
    }
    wsum[lane] = t;                                    // inclusive scan of warp totals
  }
  __syncthreads();
  const int excl = base_s + (w > 0 ? wsum[w - 1] : 0) + inc - x;
  if (v < V) seg[v] = excl;
  if (v == V - 1) seg[V] = excl + x;
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
// grid = (64-position chunks of the sorted order, 256-column slabs).  A block finds the segment
// heads (first sorted position of a token id) inside its chunk and sums each head's rows:
//   * short segments (<= 32 rows): one warp per segment, lanes own 8 columns, rows are added in
//     sorted order with 8 row loads in flight;
//   * long segments (a frequent token): the whole block, rows staged 64 at a time, warp w taking
//     rows w, w+8, ... of each stage, the 8 per-warp sums combined in warp order.
// Both orders are fixed, so the result does not depend on timing (no floating-point atomics).
constexpr int kScatChunk = 64;
constexpr int kScatShort = 32;

template <typename T>
__global__ void __launch_bounds__(256)
embed_scatter_kernel(const int* __restrict__ ids, const T* __restrict__ G, long long ldg, int Tn,
                     int d, const float* __restrict__ clip, const int* __restrict__ perm,
                     const int* __restrict__ seg, int V, float* __restrict__ out, long long ldo,
                     float beta, float scale) {
  __shared__ float part[8][kEmbedColsPerBlock];
  __shared__ int s_pos[kScatChunk];
  __shared__ float s_r[kScatChunk];
  __shared__ int s_hk[kScatChunk], s_hv[kScatChunk], s_hn[kScatChunk];
  __shared__ unsigned s_mask[2];
  const int n_valid = seg[V];
  const int kc = blockIdx.x * kScatChunk;
  if (kc >= n_valid) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;

  // ---- heads of this chunk
  int my_v = -1, my_n = 0;
  bool head = false;
  if (threadIdx.x < kScatChunk) {
    const int k = kc + threadIdx.x;
    if (k < n_valid) {
      my_v = ids[perm[k]];
      head = (k == 0) || (ids[perm[k - 1]] != my_v);
      if (head) my_n = seg[my_v + 1] - k;
    }
    const unsigned m = __ballot_sync(0xffffffffu, head);
    if (lane == 0) s_mask[w] = m;
  }
  __syncthreads();
  const int n_heads = __popc(s_mask[0]) + __popc(s_mask[1]);
  if (threadIdx.x < kScatChunk && head) {
    const int slot = (w == 1 ? __popc(s_mask[0]) : 0) + __popc(s_mask[w] & ((1u << lane) - 1u));
    s_hk[slot] = kc + threadIdx.x;
    s_hv[slot] = my_v;
    s_hn[slot] = my_n;
  }
  __syncthreads();

  const int c = blockIdx.y * kEmbedColsPerBlock + lane * 8;
  const int nvalid = min(8, d - c);
  const bool vec = ((reinterpret_cast<uintptr_t>(G) & 15) == 0) && ((ldg * sizeof(T)) % 16 == 0);
  const bool ovec = ((reinterpret_cast<uintptr_t>(out) & 15) == 0) && ((ldo & 3) == 0);

  // ---- short segments: one warp each
  for (int h = w; h < n_heads; h += 8) {
    const int n = s_hn[h];
    if (n > kScatShort || nvalid <= 0) continue;
    const int k0 = s_hk[h], v = s_hv[h];
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int b0 = 0; b0 < n; b0 += 8) {
      float vals[8][8];
      float r[8];
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if (b0 + b < n) {
          const int pos = perm[k0 + b0 + b];
          r[b] = clip[pos / Tn];
          load8<T>(G + size_t(pos) * ldg + c, nvalid, vec, vals[b]);
        } else {
          r[b] = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) vals[b][e] = 0.f;
        }
      }
#pragma unroll
      for (int b = 0; b < 8; ++b)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(r[b], vals[b][e], acc[e]);
    }
    float* o = out + size_t(v) * ldo + c;
    if (ovec && nvalid == 8) {
      float4 a = make_float4(acc[0] * scale, acc[1] * scale, acc[2] * scale, acc[3] * scale);
      float4 b = make_float4(acc[4] * scale, acc[5] * scale, acc[6] * scale, acc[7] * scale);
      if (beta != 0.f) {
        const float4 oa = *reinterpret_cast<const float4*>(o), ob = *reinterpret_cast<const float4*>(o + 4);
        a.x += oa.x; a.y += oa.y; a.z += oa.z; a.w += oa.w;
        b.x += ob.x; b.y += ob.y; b.z += ob.z; b.w += ob.w;
      }
      *reinterpret_cast<float4*>(o) = a;
      *reinterpret_cast<float4*>(o + 4) = b;
    } else {
      for (int e = 0; e < nvalid; ++e) o[e] = (beta != 0.f ? o[e] : 0.f) + acc[e] * scale;
    }
  }

  // ---- long segments: the whole block, one after another
  for (int h = 0; h < n_heads; ++h) {
    const int n = s_hn[h];
    if (n <= kScatShort) continue;
    const int k0 = s_hk[h], v = s_hv[h];
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int base = 0; base < n; base += kScatChunk) {
      const int m = min(kScatChunk, n - base);
      __syncthreads();
      if (threadIdx.x < m) {
        const int pos = perm[k0 + base + threadIdx.x];
        s_pos[threadIdx.x] = pos;
        s_r[threadIdx.x] = clip[pos / Tn];
      }
      __syncthreads();
      if (nvalid > 0) {
        float vals[kScatChunk / 8][8];
#pragma unroll
        for (int b = 0; b < kScatChunk / 8; ++b) {
          const int k = w + 8 * b;
          if (k < m) {
            load8<T>(G + size_t(s_pos[k]) * ldg + c, nvalid, vec, vals[b]);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) vals[b][e] = 0.f;
          }
        }
#pragma unroll
        for (int b = 0; b < kScatChunk / 8; ++b) {
          const int k = w + 8 * b;
          if (k < m) {
            const float r = s_r[k];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = fmaf(r, vals[b][e], acc[e]);
          }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) part[w][lane * 8 + e] = acc[e];
    __syncthreads();
    const int cc = blockIdx.y * kEmbedColsPerBlock + threadIdx.x;
    if (cc < d) {
      float sum = 0.f;
#pragma unroll
      for (int ww = 0; ww < 8; ++ww) sum += part[ww][threadIdx.x];
      float* o = out + size_t(v) * ldo + cc;
      sum *= scale;
      *o = (beta != 0.f) ? (*o + sum) : sum;
    }
    __syncthreads();
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
    embed_norm_kernel<float><<<B * slabs, kEmbedNormThreads, smem, st>>>(ids, (const float*)G, ldg, T, d, V, slabs,
                                                          partials, first_occ, dev_status);
  else
    embed_norm_kernel<__nv_bfloat16><<<B * slabs, kEmbedNormThreads, smem, st>>>(
        ids, (const __nv_bfloat16*)G, ldg, T, d, V, slabs, partials, first_occ, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_embed_sort(const int* ids, int n, int V, const EmbedSortWs& ws, int* dev_status,
                            cudaStream_t st) {
  DP_CUDA_OK(cudaMemsetAsync(ws.counts, 0, size_t(ws.chunks) * V * sizeof(int), st));
  sort_hist_kernel<<<ws.chunks, kSortChunk, 0, st>>>(ids, n, V, ws.counts, dev_status);
  DP_LAUNCH_OK();
  sort_chunk_prefix_kernel<<<ceil_div(V, 1024), 1024, 0, st>>>(ws.counts, ws.chunks, V, ws.seg,
                                                             ws.block_sums);
  DP_LAUNCH_OK();
  sort_scan_kernel<<<ceil_div(V, 1024), 1024, 0, st>>>(ws.seg, V, ws.block_sums);
  DP_LAUNCH_OK();
  sort_place_kernel<<<ws.chunks, kSortChunk, 0, st>>>(ids, n, V, ws.counts, ws.seg, ws.perm);
  DP_LAUNCH_OK();
  return DP_OK;
}

dp_status launch_embed_scatter(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int n,
                               int T, int d, int V, const float* clip, const int* perm,
                               const int* seg, float* out, int64_t ldo, float beta, float scale,
                               bool clear, cudaStream_t st) {
  // beta == 0: the table is cleared once (unless the caller already filled it, e.g. with
  // noise), then every touched row receives table + scale*sum
  if (beta == 0.f && clear) {
    DP_CUDA_OK(cudaMemset2DAsync(out, size_t(ldo) * sizeof(float), 0, size_t(d) * sizeof(float),
                                 size_t(V), st));
  }
  dim3 grid(ceil_div(n, kScatChunk), ceil_div(d, kEmbedColsPerBlock));
  if (dt == DP_F32)
    embed_scatter_kernel<float><<<grid, 256, 0, st>>>(ids, (const float*)G, ldg, T, d, clip, perm,
                                                     seg, V, out, ldo, 1.f, scale);
  else
    embed_scatter_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(ids, (const __nv_bfloat16*)G, ldg, T,
                                                             d, clip, perm, seg, V, out, ldo, 1.f,
                                                             scale);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
