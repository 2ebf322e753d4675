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
  extern __shared__ __align__(16) int sm_i[];
  const int Tp = (Tn + 3) & ~3;  // padded so that every array starts on a 16-byte boundary
  int* s_id = sm_i;              // token id, -1 if out of range
  int* s_fo = sm_i + Tp;         // first occurrence
  int* s_ord = sm_i + 2 * Tp;    // rows ordered by (first occurrence, position); sign bit = group end
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

  // First occurrence and position in the grouped order.  Tokens are ordered by (first
  // occurrence, position); a token's rank is the number of tokens ordered before it.  Inside
  // the warp's own 32-token window the ids are matched with __match_any_sync (the peers with a
  // lower lane come first); all windows are then walked once through shared memory, four ids
  // per 128-bit load, updating the earliest equal id and nothing else -- the rank needs the
  // first occurrences of ALL tokens, so it is taken in a second, equally short walk.
  const int t_round = (Tn + 31) & ~31;
  const int Tn4 = Tn & ~3;
  for (int t = threadIdx.x; t < t_round; t += blockDim.x) {
    const bool live = t < Tn;
    const int id = live ? s_id[t] : -2 - lane;             // unique sentinel for padding lanes
    const int key = (id == -1) ? -2 - 64 - lane : id;      // bad ids never match anything
    const unsigned peers = __match_any_sync(0xffffffffu, key);
    const int base = t - lane;
    int fo = base + (__ffs(peers) - 1);                    // earliest equal id in this window
    if (live && id >= 0) {
      const int4* v4 = reinterpret_cast<const int4*>(s_id);
      for (int s4 = 0; s4 < (base >> 2); ++s4) {           // windows before this one
        const int4 q = v4[s4];
        const int s = s4 << 2;
        if (q.w == id) fo = min(fo, s + 3);
        if (q.z == id) fo = min(fo, s + 2);
        if (q.y == id) fo = min(fo, s + 1);
        if (q.x == id) fo = min(fo, s);
      }
    }
    if (live) s_fo[t] = (id >= 0) ? fo : t;
  }
  __syncthreads();

  // rank of token t in the order (first occurrence, position)
  for (int t = threadIdx.x; t < Tn; t += blockDim.x) {
    const int fo = s_fo[t];
    int rank = 0;
    const int4* f4 = reinterpret_cast<const int4*>(s_fo);
    for (int s4 = 0; s4 < (Tn4 >> 2); ++s4) {
      const int4 q = f4[s4];
      const int s = s4 << 2;
      rank += (q.x < fo) || (q.x == fo && s < t);
      rank += (q.y < fo) || (q.y == fo && s + 1 < t);
      rank += (q.z < fo) || (q.z == fo && s + 2 < t);
      rank += (q.w < fo) || (q.w == fo && s + 3 < t);
    }
    for (int s = Tn4; s < Tn; ++s) {
      const int f = s_fo[s];
      rank += (f < fo) || (f == fo && s < t);
    }
    if (dp_in_range(rank, Tn, dev_status)) s_ord[rank] = t;
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
        if (r < hi && dp_in_range(t, Tn, dev_status) && s_id[t] >= 0) {
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
                  const int* __restrict__ seg, int* __restrict__ perm, int* __restrict__ dev_status) {
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
  const int dst = seg[id] + counts[size_t(chunk) * V + id] + r;
  if (dp_in_range(dst, n, dev_status)) perm[dst] = j;
}

// ------------------------------------------------------------------ segmented row sum
// The sorted order is cut into 32-position chunks; grid = (chunks, 256-column slabs).
//   pass 1 (embed_scatter_kernel): a block finds the segments (runs of one token id) that meet
//     its chunk.  Short segments (<= 32 rows) are summed by one warp each, from their head, in
//     sorted order, and written to the table.  Rows of LONG segments (a frequent token) are
//     summed per chunk by the whole block -- warp w takes rows w, w+8, ... and the eight warp
//     sums are added in warp order -- into a partial buffer [chunk][slot][column]; slot 0 is the
//     segment that continues from the previous chunk, slot 1 the one that starts in this chunk
//     (a 32-position chunk can meet at most one of each).
//   pass 2 (embed_scatter_combine_kernel): the block whose chunk holds a long segment's head
//     adds that segment's partials in chunk order and writes the table row.
// Every order is fixed, so the result does not depend on timing (no floating-point atomics),
// and a very frequent token is spread over as many blocks as it has chunks.
constexpr int kScatChunk = 32;     // sorted positions per block
constexpr int kScatShort = 32;     // longest segment handled by a single warp
constexpr int kScatBatch = 4;      // row loads in flight per lane

template <typename T>
__global__ void __launch_bounds__(256)
embed_scatter_kernel(const int* __restrict__ ids, const T* __restrict__ G, long long ldg, int Tn,
                     int d, const float* __restrict__ clip, const int* __restrict__ perm,
                     const int* __restrict__ seg, int V, float* __restrict__ out, long long ldo,
                     float beta, float scale, float* __restrict__ long_part, int n_rows,
                     int* __restrict__ dev_status) {
  __shared__ float part[8][kEmbedColsPerBlock];
  __shared__ int s_pos[kScatChunk + kScatShort];
  __shared__ float s_r[kScatChunk + kScatShort];
  __shared__ int s_hk[kScatChunk], s_hv[kScatChunk], s_hn[kScatChunk];
  __shared__ unsigned s_mask, s_long0, s_long1;
  const int n_valid = seg[V];
  const int kc = blockIdx.x * kScatChunk;
  if (kc >= n_valid) return;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;

  // ---- classify the chunk's positions (warp 0) and stage positions / clip factors of the
  //      chunk and of the kScatShort rows after it (threads 0..63)
  int my_v = -1, my_n = 0;
  bool head = false;
  if (threadIdx.x < kScatChunk) {
    const int k = kc + threadIdx.x;
    int s0 = 0;
    if (k < n_valid) {
      const int pos = perm[k];
      if (dp_in_range(pos, n_rows, dev_status)) my_v = ids[pos];
      if (dp_in_range(my_v, V, dev_status)) {
        s0 = seg[my_v];
        my_n = seg[my_v + 1] - s0;
        head = (s0 == k);
      }
    }
    const bool is_long = my_n > kScatShort;
    const unsigned m = __ballot_sync(0xffffffffu, head);
    const unsigned l0 = __ballot_sync(0xffffffffu, is_long && s0 < kc);     // continues from before
    const unsigned l1 = __ballot_sync(0xffffffffu, is_long && s0 >= kc);    // starts in this chunk
    if (lane == 0) { s_mask = m; s_long0 = l0; s_long1 = l1; }
  }
  if (threadIdx.x < kScatChunk + kScatShort) {
    const int k = kc + threadIdx.x;
    if (k < n_valid) {
      int pos = perm[k];
      if (!dp_in_range(pos, n_rows, dev_status)) pos = 0;   // checked build: flagged, row 0 stands in
      s_pos[threadIdx.x] = pos;
      s_r[threadIdx.x] = clip[pos / Tn];
    }
  }
  __syncthreads();
  const int n_heads = __popc(s_mask);
  if (threadIdx.x < kScatChunk && head) {
    const int slot = __popc(s_mask & ((1u << lane) - 1u));
    s_hk[slot] = kc + threadIdx.x;
    s_hv[slot] = my_v;
    s_hn[slot] = my_n;
  }
  __syncthreads();

  const int c = blockIdx.y * kEmbedColsPerBlock + lane * 8;
  const int nvalid = min(8, d - c);
  const bool vec = ((reinterpret_cast<uintptr_t>(G) & 15) == 0) && ((ldg * sizeof(T)) % 16 == 0);
  const bool ovec = ((reinterpret_cast<uintptr_t>(out) & 15) == 0) && ((ldo & 3) == 0);

  // ---- short segments: one warp each, rows in sorted order
  for (int h = w; h < n_heads; h += 8) {
    const int n = s_hn[h];
    if (n > kScatShort || nvalid <= 0) continue;
    const int o0 = s_hk[h] - kc, v = s_hv[h];          // rows o0 .. o0+n-1 of the staged window
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int b0 = 0; b0 < n; b0 += kScatBatch) {
      float vals[kScatBatch][8];
      float r[kScatBatch];
#pragma unroll
      for (int b = 0; b < kScatBatch; ++b) {
        if (b0 + b < n) {
          r[b] = s_r[o0 + b0 + b];
          load8<T>(G + size_t(s_pos[o0 + b0 + b]) * ldg + c, nvalid, vec, vals[b]);
        } else {
          r[b] = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) vals[b][e] = 0.f;
        }
      }
#pragma unroll
      for (int b = 0; b < kScatBatch; ++b)
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

  // ---- rows of long segments inside this chunk: per-chunk partial sums
#pragma unroll 1
  for (int slot = 0; slot < 2; ++slot) {
    const unsigned m = slot == 0 ? s_long0 : s_long1;
    if (m == 0u) continue;                               // uniform over the block
    const int a = __ffs(m) - 1, b = 32 - __clz(m);       // the rows form one run [a, b)
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    if (nvalid > 0) {
      float vals[kScatBatch][8];
#pragma unroll
      for (int j = 0; j < kScatBatch; ++j) {
        const int k = a + w + 8 * j;
        if (k < b) {
          load8<T>(G + size_t(s_pos[k]) * ldg + c, nvalid, vec, vals[j]);
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) vals[j][e] = 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < kScatBatch; ++j) {
        const int k = a + w + 8 * j;
        if (k < b) {
          const float r = s_r[k];
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[e] = fmaf(r, vals[j][e], acc[e]);
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
      long_part[(size_t(blockIdx.x) * 2 + slot) * d + cc] = sum;
    }
    __syncthreads();
  }
}

// pass 2: table row of every long segment = beta*row + scale * (its partials in chunk order)
__global__ void __launch_bounds__(256)
embed_scatter_combine_kernel(const int* __restrict__ ids, const int* __restrict__ perm,
                             const int* __restrict__ seg, int V, int d,
                             const float* __restrict__ long_part, float* __restrict__ out,
                             long long ldo, float beta, float scale, int n_rows,
                             int* __restrict__ dev_status) {
  __shared__ int s_v, s_k0, s_n;
  const int n_valid = seg[V];
  const int kc = blockIdx.x * kScatChunk;
  if (kc >= n_valid) return;
  if (threadIdx.x < 32) {                                // at most one long head per chunk
    const int k = kc + threadIdx.x;
    int v = -1, n = 0;
    bool long_head = false;
    if (k < n_valid) {
      const int pos = perm[k];
      if (dp_in_range(pos, n_rows, dev_status)) v = ids[pos];
      if (dp_in_range(v, V, dev_status)) {
        const int s0 = seg[v];
        n = seg[v + 1] - s0;
        long_head = (s0 == k) && (n > kScatShort);
      }
    }
    const unsigned m = __ballot_sync(0xffffffffu, long_head);
    if (threadIdx.x == 0) s_n = 0;
    __syncwarp();
    if (long_head) { s_v = v; s_k0 = k; s_n = n; }
    (void)m;
  }
  __syncthreads();
  const int n = s_n;
  if (n == 0) return;
  const int cc = blockIdx.y * kEmbedColsPerBlock + threadIdx.x;
  if (cc >= d) return;
  const int c0 = blockIdx.x, c1 = (s_k0 + n - 1) / kScatChunk;
  float sum = long_part[(size_t(c0) * 2 + 1) * d + cc];            // starts in its own chunk
  for (int cch = c0 + 1; cch <= c1; ++cch) sum += long_part[(size_t(cch) * 2 + 0) * d + cc];
  float* o = out + size_t(s_v) * ldo + cc;
  sum *= scale;
  *o = (beta != 0.f) ? (*o + sum) : sum;
}

}  // namespace

dp_status launch_embed_norms(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int B, int T,
                             int d, int V, float* partials, int* first_occ, int* dev_status,
                             cudaStream_t st) {
  const int slabs = ceil_div(d, kEmbedColsPerBlock);
  const size_t smem = size_t(3) * ((T + 3) & ~3) * sizeof(int);
  if (first_use_on_this_device(reinterpret_cast<const void*>(&launch_embed_norms))) {
    DP_CUDA_OK(cudaFuncSetAttribute(embed_norm_kernel<float>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    3 * kEmbedMaxT * (int)sizeof(int)));
    DP_CUDA_OK(cudaFuncSetAttribute(embed_norm_kernel<__nv_bfloat16>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    3 * kEmbedMaxT * (int)sizeof(int)));
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
  sort_place_kernel<<<ws.chunks, kSortChunk, 0, st>>>(ids, n, V, ws.counts, ws.seg, ws.perm, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

// Test hook of the checked build: one thread runs the range test on (idx, n) and touches no
// memory -- shows that an index outside its array is reported (and only in the checked build).
__global__ void bounds_probe_kernel(long long idx, long long n, int* dev_status) {
  (void)dp_in_range(idx, n, dev_status);
}
dp_status launch_bounds_probe(long long idx, long long n, int* dev_status, cudaStream_t st) {
  bounds_probe_kernel<<<1, 1, 0, st>>>(idx, n, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

size_t embed_scatter_partial_bytes(long long n, int d) {
  return align_up(size_t((n + kScatChunk - 1) / kScatChunk) * 2 * size_t(d) * sizeof(float), 256);
}

dp_status launch_embed_scatter(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int n,
                               int T, int d, int V, const float* clip, const int* perm,
                               const int* seg, float* out, int64_t ldo, float beta, float scale,
                               bool clear, float* long_part, cudaStream_t st, int* dev_status) {
  // beta == 0: the table is cleared once (unless the caller already filled it, e.g. with
  // noise), then every touched row receives table + scale*sum
  if (beta == 0.f && clear) {
    DP_CUDA_OK(cudaMemset2DAsync(out, size_t(ldo) * sizeof(float), 0, size_t(d) * sizeof(float),
                                 size_t(V), st));
  }
  dim3 grid(ceil_div(n, kScatChunk), ceil_div(d, kEmbedColsPerBlock));
  if (dt == DP_F32)
    embed_scatter_kernel<float><<<grid, 256, 0, st>>>(ids, (const float*)G, ldg, T, d, clip, perm,
                                                     seg, V, out, ldo, 1.f, scale, long_part, n,
                                                     dev_status);
  else
    embed_scatter_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(ids, (const __nv_bfloat16*)G, ldg, T,
                                                             d, clip, perm, seg, V, out, ldo, 1.f,
                                                             scale, long_part, n, dev_status);
  DP_LAUNCH_OK();
  embed_scatter_combine_kernel<<<grid, 256, 0, st>>>(ids, perm, seg, V, d, long_part, out, ldo, 1.f,
                                                     scale, n, dev_status);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
