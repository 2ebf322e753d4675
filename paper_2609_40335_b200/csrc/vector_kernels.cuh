// Launchers for bias / LayerNorm parameters (vector_kernels.cu).
#pragma once

#include "dp_common.cuh"

namespace dpg {

constexpr int kVecMaxParams = 96;      // parameters per launch (parameter-block limit)

int vector_total_slabs(const dp_vector_desc* prm, int n);
int vector_row_splits(const dp_vector_desc* prm, int n, int B, int T, int sms);

// partials: [B][n_per]; this call fills columns 0 .. vector_total_slabs-1 of every example
dp_status launch_vector_norms(const dp_vector_desc* prm, int n, dp_dtype dt, int B, int T,
                              float* partials, int n_per, cudaStream_t st);
// partial_ws: [row splits][sum of p over one launch's parameters] floats
dp_status launch_vector_sums(const dp_vector_desc* prm, int n, dp_dtype dt, int B, int T,
                             const float* clip, float* const* outs, float beta, int with_noise,
                             float amp, float scale, uint64_t seed, const uint32_t* tensor_ids,
                             uint32_t step, float* partial_ws, cudaStream_t st);

}  // namespace dpg
