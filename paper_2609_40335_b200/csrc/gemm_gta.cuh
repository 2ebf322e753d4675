// Declarations for the tensor-core G^T A kernels (clipped sum and DIRECT per-example norm).
#pragma once

#include "dp_common.cuh"
#include "fma_kernels.cuh"
#include "ghost_plan.cuh"

namespace dpg {

constexpr int kGtaMaxLayers = 80;       // layers per launch (parameter-block limit)

// Plain data: copied into kernel parameters.
struct GtaLayer {
  float* out;             // (M, N) destination when the K range is not split
  float* partial;         // [nsplit][M][N] planes when it is
  long long ldo;
  int M, N;               // p, d
  int tiles_m, tiles_n;   // 128 x 256 output tiles
  int nsplit;
  int ksteps_per_split;
  int item_begin;
  int col_begin;          // square-sum mode: first partial-sum column of this layer
  float beta;
  int prescaled;          // 1: the clip factors were applied to this layer's narrow operand beforehand
  float noise_amp;        // sigma*C of the fused noise, negative = none
  uint32_t tensor_id;     // noise stream id of this output tensor
};

// Fused Gaussian mechanism of a grouped call (host side).
struct GtaNoise {
  float amp, scale;
  uint64_t seed;
  uint32_t step;
  const uint32_t* tensor_ids;   // [n_layers]
};

int gta_choose_nsplit(const dp_linear_desc* layers, int n_layers, int B, int T, int sms);
// scratch of a grouped call behind the clip factors: K-split planes (if any) and the pre-scaled
// copies of very narrow operands
size_t gta_partial_bytes(const dp_linear_desc* layers, int n_layers, int B, int T, int sms);

// One persistent launch over the output tiles of all layers (plus split-K reduces if needed).
dp_status launch_clip_accumulate_tc(const dp_linear_desc* layers, int n_layers, int B, int T,
                                    const float* clip, float* const* outs, const int64_t* ldos,
                                    float beta, const GtaNoise* noise, float* partial_ws,
                                    int* dev_status, cudaStream_t st);

dp_status launch_direct_norm_tc(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                                float* partials, int* dev_status, cudaStream_t st);

}  // namespace dpg
