// Tensor-core cross term of a tied embedding / LM head (cross_term_tc.cu).
#pragma once

#include "dp_common.cuh"

namespace dpg {

int cross_term_tc_partials_per_example(int T);

// partials: [B][ceil(T/128)^2] floats, example-major
dp_status launch_cross_term_tc(const int* ids, const void* Ge, int64_t ldge, const void* Al,
                               int64_t ldal, const void* Gl, int64_t ldgl, int B, int T, int d, int V,
                               float* partials, int* dev_status, cudaStream_t st);

}  // namespace dpg
