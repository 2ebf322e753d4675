// Host-side work planning for dp_ghost_norms: which kernel each layer runs on, how wide
// operands are split across CTAs, and where each partial sum lands in the workspace.
#pragma once

#include <vector>

#include "dp_common.cuh"

namespace dpg {

constexpr int kGhostMaxLayers = 96;     // layers per tensor-core launch (parameter-block limit)

// Plain data: copied into kernel parameters.
struct GhostLayerPlan {
  int a_steps;       // 64-column steps over d
  int g_steps;       // 64-column steps over p
  int split_on_g;    // 1: G's columns are chunked across CTAs, 0: A's are
  int nsplit;        // number of chunks
  int chunk_steps;   // steps per chunk of the split operand
  int item_begin;    // first work item of this layer inside its launch
  int col_begin;     // first partial-sum column of this layer (per example)
};

struct DirectLayerPlan {
  int tiles_m, tiles_n;   // 128 x 256 tiles of the p x d gradient
  int col_begin;
};

struct GhostPlan {
  bool pair = false;                    // T > 128: 256 x 256 tiles on CTA pairs (two partial sums per item)
  int ntp = 0;                          // tile pairs (ti <= tj) of a T x T Gram matrix
  int n_per = 0;                        // partial sums per example over all layers
  std::vector<GhostLayerPlan> layer;    // indexed like the caller's layer array
  std::vector<DirectLayerPlan> direct;  // indexed like the caller's layer array
  std::vector<int> mode_used;           // DP_NORM_GHOST / DP_NORM_DIRECT per layer
  std::vector<int> ghost_layers;        // indices run by the Gram kernel
  std::vector<int> direct_layers;       // indices run by the gradient-tile kernel
};

// T*T > d*p selects DIRECT under AUTO (strict), otherwise GHOST.
// allow_pair = false keeps the single-CTA Gram kernel whatever T is.
GhostPlan plan_ghost_norms(const dp_linear_desc* layers, int n_layers, int B, int T, int sms,
                           bool allow_pair = true);

dp_status launch_ghost_norm_pair(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                                 float* partials, int* dev_status, cudaStream_t st);

// other_side != NULL: the second operand of every Gram product is taken from other_side[l] (same
// shapes as layers[l]) instead of layers[l] itself (the split fp32 path).
dp_status launch_ghost_norm_tc(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                               float* partials, int* dev_status, cudaStream_t st,
                               const dp_linear_desc* other_side = nullptr);

}  // namespace dpg
