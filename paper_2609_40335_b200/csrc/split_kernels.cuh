// Split of fp32 operands into two bf16 terms for the tensor-core path of DP_F32 inputs.
#pragma once

#include "dp_common.cuh"

namespace dpg {

// operand width rounded up to 8 columns (a 16-byte pitch for the TMA tensor maps)
inline int split_padded(int c) { return (c + 7) / 8 * 8; }
// bytes of ONE widened operand: rows x 3*padded(c) bf16 (column form) = B x 3T x padded(c) (row form)
inline size_t split_bytes(long long rows, int c) {
  return align_up(size_t(rows) * 3 * size_t(split_padded(c)) * 2, 256);
}

// X = [hi | hi | lo], Y = [hi | lo | hi], each (rows, 3*padded(c)) bf16
dp_status launch_split_cols(const float* src, int64_t lds, int64_t rows, int c, void* X, void* Y,
                            cudaStream_t st);
// dst (B, 3T, padded(c)): the terms {hi, hi, lo} (lo_slab 2) or {hi, lo, hi} (lo_slab 1) of
// scale[i] * src, stacked along the token axis of every example; scale may be NULL
dp_status launch_split_rows(const float* src, int64_t lds, int B, int T, int c, const float* scale,
                            int lo_slab, void* dst, cudaStream_t st);

}  // namespace dpg
