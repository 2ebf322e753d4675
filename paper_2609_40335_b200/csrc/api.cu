// extern "C" entry points: argument checks, work planning, workspace carving, launches.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <mutex>
#include <set>
#include <utility>

#include "cross_term.cuh"
#include "dp_common.cuh"
#include "fma_kernels.cuh"
#include "gemm_gta.cuh"
#include "ghost_plan.cuh"
#include "split_kernels.cuh"
#include "tma_host.cuh"
#include "vector_kernels.cuh"

namespace dpg {

int g_last_cuda_error = 0;
int g_force_fma = 0;
long long g_kernel_launches = 0;
long long g_wait_limit = 1500000000LL;
const uint32_t* g_step_dev = nullptr;
int g_ghost_single = 0;
int g_reserved_sms = 0;

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_device_mutex;
}

static int device_sm_count() {
  static int n[kMaxDevices] = {};
  int dev = 0, v = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  if (n[dev] == 0) {
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
      n[dev] = v;
    else
      return 148;          // B200; not cached so a later call can still query the device
  }
  return n[dev];
}

// SMs the persistent kernels size their grids for: all of the device's, less the ones the caller
// set aside (dp_set_reserved_sms), kept even (CTA pairs) and never below two.
int sm_count() {
  const int n = device_sm_count() - g_reserved_sms;
  return std::max(2, n & ~1);
}

bool first_use_on_this_device(const void* key) {
  static std::set<std::pair<const void*, int>> seen;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return true;     // set up again rather than never
  std::lock_guard<std::mutex> lock(g_device_mutex);
  return seen.insert(std::make_pair(key, dev)).second;
}

// ---- planning of dp_ghost_norms ------------------------------------------------------------
GhostPlan plan_ghost_norms(const dp_linear_desc* layers, int n_layers, int B, int T, int sms,
                           bool allow_pair) {
  GhostPlan plan;
  plan.pair = allow_pair && T > 128 && !g_ghost_single;
  const int nt = ceil_div(T, plan.pair ? 256 : 128);
  const int slots = plan.pair ? 2 : 1;           // partial sums per work item
  const int units = plan.pair ? sms / 2 : sms;   // persistent CTAs or CTA pairs
  plan.ntp = nt * (nt + 1) / 2;
  plan.layer.resize(n_layers);
  plan.direct.resize(n_layers);
  plan.mode_used.resize(n_layers);
  for (int l = 0; l < n_layers; ++l) {
    int mode = layers[l].mode;
    if (mode == DP_NORM_AUTO)
      mode = ((long long)T * T > (long long)layers[l].d * layers[l].p) ? DP_NORM_DIRECT : DP_NORM_GHOST;
    plan.mode_used[l] = mode;
    (mode == DP_NORM_GHOST ? plan.ghost_layers : plan.direct_layers).push_back(l);
  }
  // Column chunking of wide operands.  The per-item step budget shrinks until there are at
  // least two items per SM (or the budget bottoms out).
  int budget = 64;
  for (;;) {
    long long items = 0;
    for (int l : plan.ghost_layers) {
      GhostLayerPlan& L = plan.layer[l];
      L.a_steps = ceil_div(layers[l].d, 64);
      L.g_steps = ceil_div(layers[l].p, 64);
      const int small = std::min(L.a_steps, L.g_steps), large = std::max(L.a_steps, L.g_steps);
      L.split_on_g = L.g_steps >= L.a_steps;
      int chunk = std::max(std::max(budget - small, small), 8);
      if (small + large <= budget + budget / 2) chunk = large;
      L.nsplit = ceil_div(large, chunk);
      L.chunk_steps = ceil_div(large, L.nsplit);
      L.nsplit = ceil_div(large, L.chunk_steps);
      items += (long long)B * plan.ntp * L.nsplit;
    }
    if (items >= 2LL * units || budget <= 8 || plan.ghost_layers.empty()) break;
    budget /= 2;
  }
  // longest items first: with a static round-robin split the last, partly filled wave then
  // holds the cheapest items
  std::stable_sort(plan.ghost_layers.begin(), plan.ghost_layers.end(), [&](int a, int b) {
    auto cost = [&](int l) {
      const GhostLayerPlan& L = plan.layer[l];
      return std::min(L.a_steps, L.g_steps) + L.chunk_steps;
    };
    return cost(a) > cost(b);
  });
  int col = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (plan.mode_used[l] == DP_NORM_GHOST) {
      plan.layer[l].col_begin = col;
      plan.layer[l].item_begin = 0;
      col += plan.ntp * plan.layer[l].nsplit * slots;
    } else {
      plan.direct[l].tiles_m = ceil_div(layers[l].p, 128);
      plan.direct[l].tiles_n = ceil_div(layers[l].d, 256);
      plan.direct[l].col_begin = col;
      col += plan.direct[l].tiles_m * plan.direct[l].tiles_n;
    }
  }
  plan.n_per = col;
  return plan;
}

static bool finite_pos(float x) { return std::isfinite(x) && x > 0.f; }

static dp_status check_linear(const dp_linear_desc& L, dp_dtype dt, bool tc) {
  if (!L.A || !L.G || L.d <= 0 || L.p <= 0 || L.lda < L.d || L.ldg < L.p) return DP_ERR_INVALID_ARG;
  if (L.mode != DP_NORM_AUTO && L.mode != DP_NORM_GHOST && L.mode != DP_NORM_DIRECT)
    return DP_ERR_INVALID_ARG;
  if (tc && (!aligned16(L.A) || !aligned16(L.G) || (L.lda % 8) || (L.ldg % 8))) return DP_ERR_ALIGNMENT;
  (void)dt;
  return DP_OK;
}

// ---- fp32 inputs on the tensor cores (operands split into two bf16 terms, see split_kernels.cu)
// Taken for layers that are large enough for a tensor-core tile to pay; tiny layers (and the test
// hook dp_debug_force_fma) stay on the plain fp32 kernels.
static bool f32_on_tensor_cores(const dp_linear_desc& L, int T) {
  return !g_force_fma && T >= 32 && L.d >= 64 && L.p >= 64;
}

// One layer's widened operands inside a workspace: `a` and `g` (and, column form, their second
// sides `a2`, `g2`), then whatever the kernels need behind them.
struct SplitLayer {
  dp_linear_desc one, other;     // descriptors of the widened bf16 operands
  size_t bytes;                  // workspace taken by the operands
};

static SplitLayer split_layout(const dp_linear_desc& L, int B, int T, bool column_form, char* base) {
  SplitLayer S;
  memset(&S, 0, sizeof(S));
  const size_t na = split_bytes((long long)B * T, L.d), ng = split_bytes((long long)B * T, L.p);
  const int dp_ = split_padded(L.d), pp = split_padded(L.p);
  S.one.mode = S.other.mode = DP_NORM_GHOST;
  if (column_form) {             // (B*T, 3*padded) operands, two sides each
    S.one.A = base; S.one.G = base + na; S.other.A = base + na + ng; S.other.G = base + 2 * na + ng;
    S.one.d = S.other.d = 3 * dp_; S.one.p = S.other.p = 3 * pp;
    S.one.lda = S.other.lda = 3 * dp_; S.one.ldg = S.other.ldg = 3 * pp;
    S.bytes = 2 * (na + ng);
  } else {                       // (B, 3T, padded) operands
    S.one.A = base; S.one.G = base + na;
    S.one.d = L.d; S.one.p = L.p; S.one.lda = dp_; S.one.ldg = pp;
    S.bytes = na + ng;
  }
  return S;
}

static size_t f32_norm_ws_bytes(const dp_linear_desc& L, int B, int T, int mode, int sms) {
  const bool direct = mode == DP_NORM_DIRECT;
  SplitLayer S = split_layout(L, B, T, !direct, nullptr);
  S.one.mode = mode;
  const GhostPlan plan = plan_ghost_norms(&S.one, 1, B, direct ? 3 * T : T, sms, false);
  return S.bytes + align_up(size_t(B) * plan.n_per * sizeof(float), 256);
}

static int resolve_mode(const dp_linear_desc& L, int T) {
  if (L.mode != DP_NORM_AUTO) return L.mode;
  return ((long long)T * T > (long long)L.d * L.p) ? DP_NORM_DIRECT : DP_NORM_GHOST;
}

// norm of one fp32 layer on the tensor cores; ws holds the widened operands and the partial sums
static dp_status f32_norm_tc(const dp_linear_desc& L, int B, int T, int mode, float* sq, char* ws,
                             int* dev_status, cudaStream_t st) {
  const bool direct = mode == DP_NORM_DIRECT;
  SplitLayer S = split_layout(L, B, T, !direct, ws);
  float* partials = reinterpret_cast<float*>(ws + S.bytes);
  dp_status s;
  const float* A = static_cast<const float*>(L.A);
  const float* G = static_cast<const float*>(L.G);
  if (!direct) {
    s = launch_split_cols(A, L.lda, (int64_t)B * T, L.d, const_cast<void*>(S.one.A), const_cast<void*>(S.other.A), st);
    if (s != DP_OK) return s;
    s = launch_split_cols(G, L.ldg, (int64_t)B * T, L.p, const_cast<void*>(S.one.G), const_cast<void*>(S.other.G), st);
    if (s != DP_OK) return s;
    const GhostPlan plan = plan_ghost_norms(&S.one, 1, B, T, sm_count(), false);
    s = launch_ghost_norm_tc(&S.one, plan, B, T, partials, dev_status, st, &S.other);
    if (s != DP_OK) return s;
    return launch_reduce_partials(partials, plan.n_per, B, sq, 1.f, nullptr, st);
  }
  // DIRECT: G'^T A' per example over 3T token rows
  s = launch_split_rows(A, L.lda, B, T, L.d, nullptr, 1, const_cast<void*>(S.one.A), st);
  if (s != DP_OK) return s;
  s = launch_split_rows(G, L.ldg, B, T, L.p, nullptr, 2, const_cast<void*>(S.one.G), st);
  if (s != DP_OK) return s;
  S.one.mode = DP_NORM_DIRECT;
  const GhostPlan plan = plan_ghost_norms(&S.one, 1, B, 3 * T, sm_count(), false);
  s = launch_direct_norm_tc(&S.one, plan, B, 3 * T, partials, dev_status, st);
  if (s != DP_OK) return s;
  return launch_reduce_partials(partials, plan.n_per, B, sq, 1.f, nullptr, st);
}

}  // namespace dpg

using namespace dpg;

// Clip factors of a clip-accumulate call.  With sq given they are computed (Eq. 7) into the
// workspace and copied to `clip` if the caller wants them; with sq == NULL the caller has them
// already (dp_clip_factors / dp_clip_factors_sum) and `clip` is the input.
static dp_status resolve_clip(const float* sq, int B, float C, float* clip, float** clip_ws,
                              cudaStream_t st) {
  if (!sq) { *clip_ws = clip; return DP_OK; }
  const dp_status s = launch_clip_factors(sq, B, C, *clip_ws, nullptr, st);
  if (s != DP_OK) return s;
  if (clip) DP_CUDA_OK(cudaMemcpyAsync(clip, *clip_ws, size_t(B) * sizeof(float),
                                       cudaMemcpyDeviceToDevice, st));
  return DP_OK;
}

extern "C" {

const char* dp_status_string(dp_status s) {
  switch (s) {
    case DP_OK: return "ok";
    case DP_ERR_INVALID_ARG: return "invalid argument";
    case DP_ERR_UNSUPPORTED: return "size not supported by the built kernels";
    case DP_ERR_ALIGNMENT: return "pointer or leading dimension not aligned for TMA";
    case DP_ERR_WORKSPACE: return "workspace missing or too small";
    case DP_ERR_CUDA: return "CUDA error (see dp_last_cuda_error)";
    case DP_ERR_SCRATCH_LIMIT:
      return "problem needs more scratch than the library's built-in array holds "
             "(B * ceil(d/256) > DP_STATIC_SCRATCH_FLOATS); use dp_embed_norms with a workspace";
  }
  return "unknown status";
}

int32_t dp_last_cuda_error(void) { return g_last_cuda_error; }
const char* dp_version(void) { return "dp_ghost 0.1.0 (sm_100a)"; }
int64_t dp_kernel_launches(void) { return g_kernel_launches; }

int32_t dp_set_reserved_sms(int32_t n) {
  const int prev = g_reserved_sms;
  g_reserved_sms = std::max(0, std::min(n, device_sm_count() - 2));
  return prev;
}
int32_t dp_debug_ghost_single(int32_t on) {
  const int prev = g_ghost_single;
  g_ghost_single = on ? 1 : 0;
  return prev;
}
int64_t dp_debug_set_wait_limit(int64_t cycles) {
  const long long prev = g_wait_limit;
  g_wait_limit = cycles < 0 ? 1500000000LL : cycles;
  return prev;
}
dp_status dp_debug_noise_error_scan(float t_max, double* out3, void* stream) {
  if (!out3) return DP_ERR_INVALID_ARG;
  return launch_noise_error_scan(t_max, out3, (cudaStream_t)stream);
}
int32_t dp_debug_bounds_checked(void) { return kBoundsChecked; }
dp_status dp_debug_bounds_probe(int64_t idx, int64_t n, int32_t* dev_status, void* stream) {
  if (!dev_status) return DP_ERR_INVALID_ARG;
  return launch_bounds_probe(idx, n, dev_status, (cudaStream_t)stream);
}
int64_t dp_debug_tensor_map_encodes(void) { return tmap_encode_count(); }
int32_t dp_debug_force_fma(int32_t on) {
  const int prev = g_force_fma;
  g_force_fma = on ? 1 : 0;
  return prev;
}

// ---------------------------------------------------------------------------- ghost norms
size_t dp_ghost_norms_ws_bytes(const dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                               int32_t B, int32_t T) {
  if (!layers || n_layers <= 0 || B <= 0 || T <= 0) return 0;
  if (g_force_fma) return 0;
  if (dt == DP_F32) {            // layers run one after the other through the same workspace
    size_t need = 0;
    for (int l = 0; l < n_layers; ++l)
      if (f32_on_tensor_cores(layers[l], T))
        need = std::max(need, f32_norm_ws_bytes(layers[l], B, T, resolve_mode(layers[l], T), sm_count()));
    return need;
  }
  const GhostPlan plan = plan_ghost_norms(layers, n_layers, B, T, sm_count());
  return align_up(size_t(B) * plan.n_per * sizeof(float), 256);
}

dp_status dp_ghost_norms(dp_linear_desc* layers, int32_t n_layers, dp_dtype dt, int32_t B,
                         int32_t T, float* sq, void* ws, size_t ws_bytes, int32_t* dev_status,
                         void* stream) {
  if (!layers || n_layers <= 0 || B <= 0 || T <= 0 || !sq) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc = (dt == DP_BF16) && !g_force_fma;
  for (int l = 0; l < n_layers; ++l) {
    const dp_status s = check_linear(layers[l], dt, tc);
    if (s != DP_OK) return s;
  }
  const GhostPlan plan = plan_ghost_norms(layers, n_layers, B, T, sm_count());
  if (!tc) {
    if (dt == DP_F32 && dp_ghost_norms_ws_bytes(layers, n_layers, dt, B, T) > ws_bytes) return DP_ERR_WORKSPACE;
    for (int l = 0; l < n_layers; ++l) {
      dp_status s;
      if (dt == DP_F32 && f32_on_tensor_cores(layers[l], T)) {
        if (!ws || !aligned16(ws)) return DP_ERR_WORKSPACE;
        s = f32_norm_tc(layers[l], B, T, plan.mode_used[l], sq, static_cast<char*>(ws), dev_status, st);
      } else {
        s = launch_norms_fma(layers[l], dt, plan.mode_used[l], B, T, sq, st);
      }
      if (s != DP_OK) return s;
      layers[l].mode_used = plan.mode_used[l];
    }
    return DP_OK;
  }
  const size_t need = align_up(size_t(B) * plan.n_per * sizeof(float), 256);
  if (!ws || ws_bytes < need) return DP_ERR_WORKSPACE;
  float* partials = static_cast<float*>(ws);
  dp_status s = DP_OK;
  if (!plan.ghost_layers.empty()) {
    s = plan.pair ? launch_ghost_norm_pair(layers, plan, B, T, partials, dev_status, st)
                  : launch_ghost_norm_tc(layers, plan, B, T, partials, dev_status, st);
    if (s != DP_OK) return s;
  }
  if (!plan.direct_layers.empty()) {
    s = launch_direct_norm_tc(layers, plan, B, T, partials, dev_status, st);
    if (s != DP_OK) return s;
  }
  s = launch_reduce_partials(partials, plan.n_per, B, sq, 1.f, nullptr, st);
  if (s != DP_OK) return s;
  for (int l = 0; l < n_layers; ++l) layers[l].mode_used = plan.mode_used[l];
  return DP_OK;
}

// ------------------------------------------------------------------------ embedding norms
size_t dp_embed_norms_ws_bytes(int32_t B, int32_t T, int32_t d) {
  if (B <= 0 || T <= 0 || d <= 0) return 0;
  return align_up(size_t(B) * ceil_div(d, kEmbedColsPerBlock) * sizeof(float), 256);
}

dp_status dp_embed_norms(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt, int32_t B,
                         int32_t T, int32_t d, int32_t V, float* sq, int32_t* first_occ, void* ws,
                         size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!ids || !G || !sq || B <= 0 || T <= 0 || d <= 0 || V <= 0 || ldg < d) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  if (T > kEmbedMaxT) return DP_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < dp_embed_norms_ws_bytes(B, T, d)) return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* partials = static_cast<float*>(ws);
  dp_status s = launch_embed_norms(ids, G, ldg, dt, B, T, d, V, partials, first_occ, dev_status, st);
  if (s != DP_OK) return s;
  return launch_reduce_partials(partials, ceil_div(d, kEmbedColsPerBlock), B, sq, 1.f, nullptr, st);
}

// ------------------------------------------------------------------------ tied cross term
size_t dp_tied_cross_term_ws_bytes(int32_t B, int32_t T, int32_t d, int32_t V) {
  (void)d; (void)V;
  if (B <= 0 || T <= 0) return 0;
  // enough for either kernel: one partial per 16-token slab (fp32 path) or per 128 x 128 tile
  const int per = std::max(ceil_div(T, 16), cross_term_tc_partials_per_example(T));
  return align_up(size_t(B) * per * sizeof(float), 256);
}

dp_status dp_tied_cross_term(const int32_t* ids, const void* G_emb, int64_t ldge, const void* A_lm,
                             int64_t ldal, const void* G_lm, int64_t ldgl, dp_dtype dt, int32_t B,
                             int32_t T, int32_t d, int32_t V, float* sq, float* cross, void* ws,
                             size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!ids || !G_emb || !A_lm || !G_lm || B <= 0 || T <= 0 || d <= 0 || V <= 0)
    return DP_ERR_INVALID_ARG;
  if (!sq && !cross) return DP_ERR_INVALID_ARG;
  if (ldge < d || ldal < d || ldgl < V) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  const bool tc = (dt == DP_BF16) && !g_force_fma;
  if (tc && (!aligned16(G_emb) || !aligned16(A_lm) || (ldge % 8) || (ldal % 8))) return DP_ERR_ALIGNMENT;
  if (!ws || ws_bytes < dp_tied_cross_term_ws_bytes(B, T, d, V)) return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* partials = static_cast<float*>(ws);
  dp_status s;
  int per;
  if (tc) {
    s = launch_cross_term_tc(ids, G_emb, ldge, A_lm, ldal, G_lm, ldgl, B, T, d, V, partials,
                             dev_status, st);
    per = cross_term_tc_partials_per_example(T);
  } else {
    s = launch_cross_term_fma(ids, G_emb, ldge, A_lm, ldal, G_lm, ldgl, dt, B, T, d, V, partials,
                              dev_status, st);
    per = ceil_div(T, 16);
  }
  if (s != DP_OK) return s;
  return launch_reduce_partials(partials, per, B, sq, 2.f, cross, st);
}

// ------------------------------------------------------- bias / LayerNorm parameters
static dp_status check_vectors(const dp_vector_desc* prm, int32_t n, int32_t B, int32_t T) {
  if (!prm || n <= 0 || B <= 0 || T <= 0) return DP_ERR_INVALID_ARG;
  for (int k = 0; k < n; ++k) {
    if (!prm[k].G || prm[k].p <= 0 || prm[k].ldg < prm[k].p) return DP_ERR_INVALID_ARG;
    if (prm[k].X && prm[k].ldx < prm[k].p) return DP_ERR_INVALID_ARG;
  }
  return DP_OK;
}

size_t dp_vector_norms_ws_bytes(const dp_vector_desc* prm, int32_t n, int32_t B, int32_t T) {
  if (check_vectors(prm, n, B, T) != DP_OK) return 0;
  return align_up(size_t(B) * vector_total_slabs(prm, n) * sizeof(float), 256);
}

dp_status dp_vector_norms(const dp_vector_desc* prm, int32_t n, dp_dtype dt, int32_t B, int32_t T,
                          float* sq, void* ws, size_t ws_bytes, void* stream) {
  const dp_status c = check_vectors(prm, n, B, T);
  if (c != DP_OK) return c;
  if (!sq || (dt != DP_F32 && dt != DP_BF16)) return DP_ERR_INVALID_ARG;
  if (!ws || ws_bytes < dp_vector_norms_ws_bytes(prm, n, B, T)) return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* partials = static_cast<float*>(ws);
  const int n_per = vector_total_slabs(prm, n);
  dp_status s = launch_vector_norms(prm, n, dt, B, T, partials, n_per, st);
  if (s != DP_OK) return s;
  return launch_reduce_partials(partials, n_per, B, sq, 1.f, nullptr, st);
}

static size_t vector_partial_bytes(const dp_vector_desc* prm, int32_t n, int32_t B, int32_t T) {
  size_t worst = 0;
  for (int n0 = 0; n0 < n; n0 += kVecMaxParams) {
    const int n1 = std::min(n, n0 + kVecMaxParams);
    size_t cols = 0;
    for (int k = n0; k < n1; ++k) cols += size_t(prm[k].p);
    worst = std::max(worst, cols * vector_row_splits(prm + n0, n1 - n0, B, T, sm_count()));
  }
  return align_up(worst * sizeof(float), 256);
}

size_t dp_clip_accumulate_vectors_ws_bytes(const dp_vector_desc* prm, int32_t n, int32_t B,
                                           int32_t T) {
  if (check_vectors(prm, n, B, T) != DP_OK) return 0;
  return align_up(size_t(B) * sizeof(float), 256) + vector_partial_bytes(prm, n, B, T);
}

dp_status dp_clip_accumulate_vectors(const dp_vector_desc* prm, int32_t n, dp_dtype dt, int32_t B,
                                     int32_t T, const float* sq, float C, float* clip,
                                     float* const* outs, float beta, int32_t with_noise, float sigma,
                                     float scale, uint64_t seed, const uint32_t* tensor_ids,
                                     uint32_t step, void* ws, size_t ws_bytes, void* stream) {
  const dp_status c = check_vectors(prm, n, B, T);
  if (c != DP_OK) return c;
  if ((!sq && !clip) || !outs || (dt != DP_F32 && dt != DP_BF16)) return DP_ERR_INVALID_ARG;
  if (!(beta == 0.f || beta == 1.f) || !finite_pos(C)) return DP_ERR_INVALID_ARG;
  for (int k = 0; k < n; ++k) if (!outs[k]) return DP_ERR_INVALID_ARG;
  if (with_noise && (!tensor_ids || !std::isfinite(sigma) || sigma < 0.f || !std::isfinite(scale)))
    return DP_ERR_INVALID_ARG;
  if (!ws || ws_bytes < dp_clip_accumulate_vectors_ws_bytes(prm, n, B, T)) return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* clip_ws = static_cast<float*>(ws);
  dp_status s = resolve_clip(sq, B, C, clip, &clip_ws, st);
  if (s != DP_OK) return s;
  float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) +
                                            align_up(size_t(B) * sizeof(float), 256));
  return launch_vector_sums(prm, n, dt, B, T, clip_ws, outs, beta, with_noise ? 1 : 0, sigma * C,
                            with_noise ? scale : 1.f, seed, tensor_ids, step, partial, st);
}

// --------------------------------------------------------------------------- clip factors
dp_status dp_clip_factors_sum(float* sq, const float* sq_extra, int32_t B, float C, float* clip,
                              float* norms, void* stream) {
  if (!sq || !sq_extra || B <= 0 || !finite_pos(C)) return DP_ERR_INVALID_ARG;
  return launch_clip_factors(sq, B, C, clip, norms, (cudaStream_t)stream, sq_extra, sq);
}

dp_status dp_clip_factors(const float* sq, int32_t B, float C, float* clip, float* norms,
                          void* stream) {
  if (!sq || B <= 0 || (!clip && !norms) || !finite_pos(C)) return DP_ERR_INVALID_ARG;
  return launch_clip_factors(sq, B, C, clip, norms, (cudaStream_t)stream);
}

// ------------------------------------------------------------------------ clip accumulate
size_t dp_clip_accumulate_grouped_ws_bytes(const dp_linear_desc* layers, int32_t n_layers,
                                           dp_dtype dt, int32_t B, int32_t T) {
  if (!layers || n_layers <= 0 || B <= 0 || T <= 0) return 0;
  size_t n = align_up(size_t(B) * sizeof(float), 256);          // clip factors
  if (dt == DP_BF16 && !g_force_fma) n += gta_partial_bytes(layers, n_layers, B, T, sm_count());
  if (dt == DP_F32) {            // widened operands of one layer at a time + its K-split planes
    size_t need = 0;
    for (int l = 0; l < n_layers; ++l)
      if (f32_on_tensor_cores(layers[l], T)) {
        SplitLayer S = split_layout(layers[l], B, T, false, nullptr);
        need = std::max(need, S.bytes + gta_partial_bytes(&S.one, 1, B, 3 * T, sm_count()));
      }
    n += need;
  }
  return n;
}

static dp_status clip_accumulate_impl(const dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                                      int32_t B, int32_t T, const float* sq, float C, float* clip,
                                      float* const* outs, const int64_t* ldos, float beta,
                                      const GtaNoise* noise, void* ws, size_t ws_bytes,
                                      int32_t* dev_status, void* stream) {
  if (!layers || n_layers <= 0 || !outs || !ldos || (!sq && !clip) || B <= 0 || T <= 0) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  if (!(beta == 0.f || beta == 1.f) || !finite_pos(C)) return DP_ERR_INVALID_ARG;
  const bool tc = (dt == DP_BF16) && !g_force_fma;
  for (int l = 0; l < n_layers; ++l) {
    dp_linear_desc one = layers[l];
    one.mode = DP_NORM_AUTO;
    const dp_status s = check_linear(one, dt, tc);
    if (s != DP_OK) return s;
    if (!outs[l] || ldos[l] < layers[l].d) return DP_ERR_INVALID_ARG;
  }
  if (!ws || ws_bytes < dp_clip_accumulate_grouped_ws_bytes(layers, n_layers, dt, B, T))
    return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  float* clip_ws = static_cast<float*>(ws);
  dp_status s = resolve_clip(sq, B, C, clip, &clip_ws, st);
  if (s != DP_OK) return s;
  if (!tc) {
    char* split_ws = static_cast<char*>(ws) + align_up(size_t(B) * sizeof(float), 256);
    for (int l = 0; l < n_layers; ++l) {
      if (dt == DP_F32 && f32_on_tensor_cores(layers[l], T)) {
        // R_i multiplies G in fp32 before the split, so the GEMM runs unscaled (clip = NULL)
        SplitLayer S = split_layout(layers[l], B, T, false, split_ws);
        s = launch_split_rows(static_cast<const float*>(layers[l].A), layers[l].lda, B, T, layers[l].d,
                              nullptr, 1, const_cast<void*>(S.one.A), st);
        if (s != DP_OK) return s;
        s = launch_split_rows(static_cast<const float*>(layers[l].G), layers[l].ldg, B, T, layers[l].p,
                              clip_ws, 2, const_cast<void*>(S.one.G), st);
        if (s != DP_OK) return s;
        GtaNoise one_noise;
        if (noise) { one_noise = *noise; one_noise.tensor_ids = noise->tensor_ids + l; }
        s = launch_clip_accumulate_tc(&S.one, 1, B, 3 * T, nullptr, outs + l, ldos + l, beta,
                                      noise ? &one_noise : nullptr,
                                      reinterpret_cast<float*>(split_ws + S.bytes), dev_status, st);
        if (s != DP_OK) return s;
        continue;
      }
      s = launch_clip_accumulate_fma(layers[l].A, layers[l].lda, layers[l].G, layers[l].ldg, dt, B, T,
                                     layers[l].d, layers[l].p, clip_ws, outs[l], ldos[l], beta, st);
      if (s != DP_OK) return s;
      if (noise) {
        s = launch_add_noise(outs[l], layers[l].p, layers[l].d, ldos[l], false, noise->amp,
                             noise->scale, noise->seed, noise->tensor_ids[l], noise->step, st);
        if (s != DP_OK) return s;
      }
    }
    return DP_OK;
  }
  float* partial = reinterpret_cast<float*>(static_cast<char*>(ws) +
                                            align_up(size_t(B) * sizeof(float), 256));
  return launch_clip_accumulate_tc(layers, n_layers, B, T, clip_ws, outs, ldos, beta, noise, partial,
                                   dev_status, st);
}

dp_status dp_clip_accumulate_grouped(const dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                                     int32_t B, int32_t T, const float* sq, float C, float* clip,
                                     float* const* outs, const int64_t* ldos, float beta, void* ws,
                                     size_t ws_bytes, int32_t* dev_status, void* stream) {
  return clip_accumulate_impl(layers, n_layers, dt, B, T, sq, C, clip, outs, ldos, beta, nullptr, ws,
                              ws_bytes, dev_status, stream);
}

static bool noise_args_ok(float sigma, float C, float scale) {
  return std::isfinite(sigma) && sigma >= 0.f && finite_pos(C) && std::isfinite(scale);
}

dp_status dp_clip_accumulate_noise_grouped(const dp_linear_desc* layers, int32_t n_layers,
                                           dp_dtype dt, int32_t B, int32_t T, const float* sq,
                                           float C, float* clip, float* const* outs,
                                           const int64_t* ldos, float beta, float sigma, float scale,
                                           uint64_t seed, const uint32_t* tensor_ids, uint32_t step,
                                           void* ws, size_t ws_bytes, int32_t* dev_status,
                                           void* stream) {
  if (!tensor_ids || !noise_args_ok(sigma, C, scale)) return DP_ERR_INVALID_ARG;
  const GtaNoise noise{sigma * C, scale, seed, step, tensor_ids};
  return clip_accumulate_impl(layers, n_layers, dt, B, T, sq, C, clip, outs, ldos, beta, &noise, ws,
                              ws_bytes, dev_status, stream);
}

static dp_linear_desc one_layer(const void* A, int64_t lda, const void* G, int64_t ldg, int32_t d,
                                int32_t p) {
  dp_linear_desc L;
  L.A = A; L.lda = lda; L.d = d; L.G = G; L.ldg = ldg; L.p = p;
  L.mode = DP_NORM_AUTO; L.mode_used = 0;
  return L;
}

size_t dp_clip_accumulate_ws_bytes(dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t p) {
  if (B <= 0 || T <= 0 || d <= 0 || p <= 0) return 0;
  const dp_linear_desc L = one_layer(nullptr, d, nullptr, p, d, p);
  return dp_clip_accumulate_grouped_ws_bytes(&L, 1, dt, B, T);
}

dp_status dp_clip_accumulate(const void* A, int64_t lda, const void* G, int64_t ldg, dp_dtype dt,
                             int32_t B, int32_t T, int32_t d, int32_t p, const float* sq, float C,
                             float* clip, float* out, int64_t ldo, float beta, void* ws,
                             size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!A || !G || !out || d <= 0 || p <= 0) return DP_ERR_INVALID_ARG;
  const dp_linear_desc L = one_layer(A, lda, G, ldg, d, p);
  float* outs[1] = {out};
  const int64_t ldos[1] = {ldo};
  return dp_clip_accumulate_grouped(&L, 1, dt, B, T, sq, C, clip, outs, ldos, beta, ws, ws_bytes,
                                    dev_status, stream);
}

// ------------------------------------------------------------------ clip accumulate, embedding
static void embed_ws_layout(int B, int T, int d, int V, size_t* off_clip, size_t* off_counts,
                            size_t* off_seg, size_t* off_perm, size_t* off_blk, size_t* off_part,
                            size_t* total, int* chunks) {
  const size_t n = size_t(B) * T;
  *chunks = int((n + kSortChunk - 1) / kSortChunk);
  size_t o = 0;
  *off_clip = o;   o += align_up(size_t(B) * sizeof(float), 256);
  *off_counts = o; o += align_up(size_t(*chunks) * V * sizeof(int), 256);
  *off_seg = o;    o += align_up(size_t(V + 1) * sizeof(int), 256);
  *off_perm = o;   o += align_up(n * sizeof(int), 256);
  *off_blk = o;    o += align_up(size_t(ceil_div(V, 1024)) * sizeof(int), 256);
  *off_part = o;   o += embed_scatter_partial_bytes((long long)n, d);
  *total = o;
}

size_t dp_clip_accumulate_embed_ws_bytes(int32_t B, int32_t T, int32_t d, int32_t V) {
  if (B <= 0 || T <= 0 || V <= 0 || d <= 0) return 0;
  size_t a, b, c, e, f, g, total; int chunks;
  embed_ws_layout(B, T, d, V, &a, &b, &c, &e, &f, &g, &total, &chunks);
  return total;
}

struct EmbedNoise { float amp, scale; uint64_t seed; uint32_t tensor_id, step; };

static dp_status clip_accumulate_embed_impl(const int32_t* ids, const void* G, int64_t ldg,
                                            dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t V,
                                            const float* sq, float C, float* clip, float* out,
                                            int64_t ldo, float beta, const EmbedNoise* noise,
                                            int32_t* perm, int32_t* seg, void* ws, size_t ws_bytes,
                                            int32_t* dev_status, void* stream,
                                            const int32_t* perm_in = nullptr,
                                            const int32_t* seg_in = nullptr) {
  if (!ids || !G || (!sq && !clip) || !out || B <= 0 || T <= 0 || d <= 0 || V <= 0) return DP_ERR_INVALID_ARG;
  if ((perm_in == nullptr) != (seg_in == nullptr)) return DP_ERR_INVALID_ARG;
  if (ldg < d || ldo < d) return DP_ERR_INVALID_ARG;
  if (dt != DP_F32 && dt != DP_BF16) return DP_ERR_INVALID_ARG;
  if (!(beta == 0.f || beta == 1.f) || !finite_pos(C)) return DP_ERR_INVALID_ARG;
  if ((long long)B * T > 0x7fffffffLL) return DP_ERR_UNSUPPORTED;
  size_t o_clip, o_counts, o_seg, o_perm, o_blk, o_part, total; int chunks;
  embed_ws_layout(B, T, d, V, &o_clip, &o_counts, &o_seg, &o_perm, &o_blk, &o_part, &total, &chunks);
  if (!ws || ws_bytes < total) return DP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* w = static_cast<char*>(ws);
  float* clip_ws = reinterpret_cast<float*>(w + o_clip);
  EmbedSortWs sw;
  sw.counts = reinterpret_cast<int*>(w + o_counts);
  sw.seg = reinterpret_cast<int*>(w + o_seg);
  sw.perm = reinterpret_cast<int*>(w + o_perm);
  sw.block_sums = reinterpret_cast<int*>(w + o_blk);
  sw.chunks = chunks;
  const int n = B * T;
  dp_status s = resolve_clip(sq, B, C, clip, &clip_ws, st);
  if (s != DP_OK) return s;
  if (perm_in) {                         // sorted earlier by dp_embed_sort
    sw.perm = const_cast<int*>(perm_in);
    sw.seg = const_cast<int*>(seg_in);
  } else {
    s = launch_embed_sort(ids, n, V, sw, dev_status, st);
    if (s != DP_OK) return s;
  }
  if (perm) DP_CUDA_OK(cudaMemcpyAsync(perm, sw.perm, size_t(n) * sizeof(int),
                                       cudaMemcpyDeviceToDevice, st));
  if (seg) DP_CUDA_OK(cudaMemcpyAsync(seg, sw.seg, size_t(V + 1) * sizeof(int),
                                      cudaMemcpyDeviceToDevice, st));
  // With noise and beta == 0 the table is filled with scale*sigma*C*z (write only) in place of
  // the zero fill; with beta == 1 the noise was already drawn by whoever wrote the table first.
  bool clear = true;
  float scale = 1.f;
  if (noise) {
    scale = noise->scale;
    if (beta == 0.f) {
      s = launch_add_noise(out, V, d, ldo, true, noise->amp, noise->scale, noise->seed,
                           noise->tensor_id, noise->step, st);
      if (s != DP_OK) return s;
      clear = false;
    }
  }
  return launch_embed_scatter(ids, G, ldg, dt, n, T, d, V, clip_ws, sw.perm, sw.seg, out, ldo, beta,
                              scale, clear, reinterpret_cast<float*>(w + o_part), st, dev_status);
}

dp_status dp_clip_accumulate_embed(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                   int32_t B, int32_t T, int32_t d, int32_t V, const float* sq,
                                   float C, float* clip, float* out, int64_t ldo, float beta,
                                   int32_t* perm, int32_t* seg, void* ws, size_t ws_bytes,
                                   int32_t* dev_status, void* stream) {
  return clip_accumulate_embed_impl(ids, G, ldg, dt, B, T, d, V, sq, C, clip, out, ldo, beta, nullptr,
                                    perm, seg, ws, ws_bytes, dev_status, stream);
}

size_t dp_embed_sort_ws_bytes(int32_t B, int32_t T, int32_t V) {
  if (B <= 0 || T <= 0 || V <= 0) return 0;
  const size_t chunks = (size_t(B) * T + kSortChunk - 1) / kSortChunk;
  return align_up(chunks * V * sizeof(int), 256) + align_up(size_t(ceil_div(V, 1024)) * sizeof(int), 256);
}

dp_status dp_embed_sort(const int32_t* ids, int32_t B, int32_t T, int32_t V, int32_t* perm,
                        int32_t* seg, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!ids || !perm || !seg || B <= 0 || T <= 0 || V <= 0) return DP_ERR_INVALID_ARG;
  if ((long long)B * T > 0x7fffffffLL) return DP_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < dp_embed_sort_ws_bytes(B, T, V)) return DP_ERR_WORKSPACE;
  const int n = B * T;
  EmbedSortWs sw;
  sw.chunks = (n + kSortChunk - 1) / kSortChunk;
  sw.counts = static_cast<int*>(ws);
  sw.block_sums = reinterpret_cast<int*>(static_cast<char*>(ws) +
                                         align_up(size_t(sw.chunks) * V * sizeof(int), 256));
  sw.seg = seg;
  sw.perm = perm;
  return launch_embed_sort(ids, n, V, sw, dev_status, (cudaStream_t)stream);
}

dp_status dp_clip_accumulate_embed_sorted(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                          int32_t B, int32_t T, int32_t d, int32_t V, const float* sq,
                                          float C, float* clip, float* out, int64_t ldo, float beta,
                                          const int32_t* perm, const int32_t* seg, void* ws,
                                          size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!perm || !seg) return DP_ERR_INVALID_ARG;
  return clip_accumulate_embed_impl(ids, G, ldg, dt, B, T, d, V, sq, C, clip, out, ldo, beta, nullptr,
                                    nullptr, nullptr, ws, ws_bytes, dev_status, stream, perm, seg);
}

dp_status dp_clip_accumulate_embed_noise(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                         int32_t B, int32_t T, int32_t d, int32_t V, const float* sq,
                                         float C, float* clip, float* out, int64_t ldo, float beta,
                                         float sigma, float scale, uint64_t seed, uint32_t tensor_id,
                                         uint32_t step, int32_t* perm, int32_t* seg, void* ws,
                                         size_t ws_bytes, int32_t* dev_status, void* stream) {
  if (!noise_args_ok(sigma, C, scale)) return DP_ERR_INVALID_ARG;
  const EmbedNoise noise{sigma * C, scale, seed, tensor_id, step};
  return clip_accumulate_embed_impl(ids, G, ldg, dt, B, T, d, V, sq, C, clip, out, ldo, beta, &noise,
                                    perm, seg, ws, ws_bytes, dev_status, stream);
}

// ----------------------------------------------------------------------------------- noise
dp_status dp_add_noise(float* out, int64_t n, float sigma, float C, float scale, uint64_t seed,
                       uint32_t tensor_id, uint32_t step, void* stream) {
  if (!out || n < 0) return DP_ERR_INVALID_ARG;
  if (!std::isfinite(sigma) || sigma < 0.f || !finite_pos(C) || !std::isfinite(scale))
    return DP_ERR_INVALID_ARG;
  if (!aligned16(out)) return DP_ERR_ALIGNMENT;
  // a flat buffer is the (n, 1) tensor with pitch 1
  return launch_add_noise(out, n, 1, 1, false, sigma * C, scale, seed, tensor_id, step,
                          (cudaStream_t)stream);
}

dp_status dp_add_noise_slice(float* out, int64_t n, int64_t first_element, float sigma, float C,
                             float scale, uint64_t seed, uint32_t tensor_id, uint32_t step,
                             void* stream) {
  if (!out || n < 0 || first_element < 0) return DP_ERR_INVALID_ARG;
  if (!noise_args_ok(sigma, C, scale)) return DP_ERR_INVALID_ARG;
  if (!aligned16(out) || (first_element & 3)) return DP_ERR_ALIGNMENT;   // whole Philox counters
  return launch_add_noise(out, n, 1, 1, false, sigma * C, scale, seed, tensor_id, step,
                          (cudaStream_t)stream, first_element >> 2);
}

dp_status dp_noise_step_device(const uint32_t* dev_counter) {
  g_step_dev = dev_counter;
  return DP_OK;
}

dp_status dp_fill_noise(float* out, int64_t n, float sigma, float C, float scale, uint64_t seed,
                        uint32_t tensor_id, uint32_t step, void* stream) {
  if (!out || n < 0) return DP_ERR_INVALID_ARG;
  if (!noise_args_ok(sigma, C, scale)) return DP_ERR_INVALID_ARG;
  if (!aligned16(out)) return DP_ERR_ALIGNMENT;
  return launch_add_noise(out, n, 1, 1, true, sigma * C, scale, seed, tensor_id, step,
                          (cudaStream_t)stream);
}

}  // extern "C"
