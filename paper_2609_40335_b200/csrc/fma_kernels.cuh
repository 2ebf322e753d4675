// Declarations of the fp32-FMA launchers (fma_kernels.cu), the embedding launchers
// (embed_kernels.cu) and the noise launcher (noise_kernel.cu).
#pragma once

#include "dp_common.cuh"

namespace dpg {

dp_status launch_norms_fma(const dp_linear_desc& L, dp_dtype dt, int mode, int B, int T, float* sq,
                           cudaStream_t st);
dp_status launch_clip_accumulate_fma(const void* A, int64_t lda, const void* G, int64_t ldg,
                                     dp_dtype dt, int B, int T, int d, int p, const float* clip,
                                     float* out, int64_t ldo, float beta, cudaStream_t st);
// partials: [B * ceil(T/16)] floats, example-major
dp_status launch_cross_term_fma(const int* ids, const void* Ge, int64_t ldge, const void* Al,
                                int64_t ldal, const void* Gl, int64_t ldgl, dp_dtype dt, int B,
                                int T, int d, int V, float* partials, int* dev_status,
                                cudaStream_t st);
dp_status launch_clip_factors(const float* sq, int B, float C, float* clip, float* norms,
                              cudaStream_t st, const float* extra = nullptr,
                              float* sq_out = nullptr);

// embedding
constexpr int kEmbedMaxT = 4096;
constexpr int kEmbedColsPerBlock = 256;
dp_status launch_embed_norms(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int B, int T,
                             int d, int V, float* partials, int* first_occ, int* dev_status,
                             cudaStream_t st);
struct EmbedSortWs {
  int* counts;      // [chunks][V]   per-chunk histograms, then exclusive prefix over chunks
  int* seg;         // [V+1]
  int* perm;        // [B*T]
  int* block_sums;  // scan scratch
  int chunks;
};
constexpr int kSortChunk = 1024;
dp_status launch_embed_sort(const int* ids, int n, int V, const EmbedSortWs& ws, int* dev_status,
                            cudaStream_t st);
dp_status launch_embed_scatter(const int* ids, const void* G, int64_t ldg, dp_dtype dt, int n,
                               int T, int d, int V, const float* clip, const int* perm,
                               const int* seg, float* out, int64_t ldo, float beta, float scale,
                               bool clear, float* long_part, cudaStream_t st,
                               int* dev_status = nullptr);
dp_status launch_bounds_probe(long long idx, long long n, int* dev_status, cudaStream_t st);
// bytes of the per-chunk partial sums of long segments: [chunks][2][d] floats
size_t embed_scatter_partial_bytes(long long n, int d);

// logical (rows, cols) tensor with row pitch ld; element j = row*cols + col of the stream.
// fill: write scale*amp*z without reading out.
dp_status launch_add_noise(float* out, long long rows, int cols, long long ld, bool fill, float amp,
                           float scale, uint64_t seed, uint32_t tensor_id, uint32_t step,
                           cudaStream_t st, long long first_quad = 0);

dp_status launch_noise_error_scan(float t_max, double* out3, cudaStream_t st);

}  // namespace dpg
