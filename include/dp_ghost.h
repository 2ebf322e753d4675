/*
 * dp_ghost.h -- C ABI of the DP-SGD ghost-clipping hot path for NVIDIA B200 (sm_100a).
 *
 * What the library computes (paper: "DP-SGD", Eq. 2 and Eq. 3; "Ghost Clipping
 * Mechanism", Eq. 4 - Eq. 7; "Corrected Ghost Norm for Tied Embeddings", Eq. 11 - Eq. 13):
 *
 *   1. per-example squared gradient norms, without materialising per-example gradients,
 *      summed over the parameter blocks handed in (Eq. 6):
 *        linear layer      sq[i] += || G_i^T A_i ||_F^2 = sum_{t,s} (a_t.a_s)(g_t.g_s)
 *        embedding table   sq[i] += sum_{t,s} [id_t == id_s] (g_t.g_s)
 *        tied cross term   sq[i] += 2 <g_in_i, g_out_i>                     (Eq. 11)
 *   2. clip coefficients  R_i = min(1, C / sqrt(sq[i]))                     (Eq. 2, Eq. 7)
 *   3. the clipped sum    sum_i R_i g_i  per parameter tensor               (inner sum of Eq. 3)
 *   4. Gaussian noise     out = scale * (out + sigma*C*z), z ~ N(0, I)      (Eq. 3)
 *
 * Conventions
 *   - Every pointer marked [dev] is CUDA device memory of the current device, owned by the
 *     caller; [host] is ordinary host memory.  The library never allocates, frees or
 *     synchronises: work is enqueued on `stream` (a cudaStream_t passed as void*) and the
 *     call returns.  Scratch comes from a caller-provided [dev] workspace whose minimum
 *     size the matching *_ws_bytes function reports (0 means none is needed).
 *   - Tensors are row-major with an explicit leading dimension (elements between rows).
 *     Activations A are (B*T, d), output gradients G are (B*T, p); example i owns rows
 *     i*T .. i*T+T-1.  dp_dtype names the storage type of A / G; accumulation is fp32.
 *   - DP_BF16 tensors feed TMA: base pointers 16-byte aligned and leading dimensions a
 *     multiple of 8 elements, else DP_ERR_ALIGNMENT (no slower substitute path is taken).
 *     The logical width may be anything (V = 50257 with ld = 50264 is fine); columns past
 *     the logical width are never read.
 *   - Norm functions ADD into sq; the caller zeroes sq once per step.
 *   - `dev_status` [dev, int32, may be NULL] collects device-side problems by bitwise OR:
 *     DP_DEV_BAD_ID (a token id outside [0,V): that token is skipped), DP_DEV_BOUNDS (checked
 *     build only: a computed index fell outside its array and the access was skipped) and DP_DEV_TIMEOUT
 *     (a bounded barrier wait gave up: the launch's results are invalid).  The caller
 *     zeroes it and reads it after its own synchronisation.
 *   - Return value: DP_OK or an error found BEFORE anything was enqueued, except
 *     DP_ERR_CUDA (a launch failed; see dp_last_cuda_error).  Nothing aborts or throws.
 *   - Results are deterministic: the same inputs give bitwise-equal outputs.
 */
#ifndef DP_GHOST_H_
#define DP_GHOST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DP_OK = 0,
  DP_ERR_INVALID_ARG = 1,   /* null required pointer, non-positive size, bad enum, bad scalar */
  DP_ERR_UNSUPPORTED = 2,   /* a size beyond what the kernels were built for */
  DP_ERR_ALIGNMENT = 3,     /* pointer / leading dimension breaks the TMA rules above */
  DP_ERR_WORKSPACE = 4,     /* ws is NULL or smaller than *_ws_bytes reports */
  DP_ERR_CUDA = 5,          /* CUDA runtime / driver error; dp_last_cuda_error() has the code */
  DP_ERR_SCRATCH_LIMIT = 6  /* dp_embed_norms_static: problem larger than the built-in scratch */
} dp_status;

typedef enum { DP_F32 = 0, DP_BF16 = 1 } dp_dtype;

/* How a linear layer's per-example norm is evaluated.  GHOST forms the two T x T Gram
 * matrices A_i A_i^T and G_i G_i^T and their Frobenius inner product; DIRECT forms the
 * p x d gradient tile by tile on chip (never in memory) and sums its squares.  AUTO picks
 * DIRECT iff T*T > d*p, else GHOST. */
typedef enum { DP_NORM_AUTO = 0, DP_NORM_GHOST = 1, DP_NORM_DIRECT = 2 } dp_norm_mode;

enum { DP_DEV_BAD_ID = 1, DP_DEV_TIMEOUT = 2, DP_DEV_BOUNDS = 4 };

/* One linear layer d -> p as seen by the backward pass (Eq. 4: a_i and delta_i). */
typedef struct {
  const void* A;       /* [dev] (B*T, d) layer input */
  int64_t lda;
  int32_t d;
  const void* G;       /* [dev] (B*T, p) gradient w.r.t. the layer output */
  int64_t ldg;
  int32_t p;
  int32_t mode;        /* in : dp_norm_mode */
  int32_t mode_used;   /* out: DP_NORM_GHOST or DP_NORM_DIRECT, what was enqueued */
} dp_linear_desc;

/* ---- per-example norms of linear layers (Eq. 4 - Eq. 6; LM head = a layer with p = V) ----
 * layers [host, n_layers entries, mode_used written back]; sq [dev, B floats, +=].
 * All layers share B, T and dt.  DP_BF16 runs on tcgen05 tensor cores.  DP_F32 layers with
 * T >= 32 and d, p >= 64 run there too: every fp32 operand is split into two bf16 terms in the
 * workspace (x = hi + lo up to 2^-17) and each product is taken as hi*hi' + hi*lo' + lo*hi' with
 * fp32 accumulation -- about 1e-5 relative, inside the 1e-4 of fp32 inputs; it needs a workspace of
 * about three times the layer's inputs (dp_ghost_norms_ws_bytes says how much; layers run one after
 * the other through it).  Smaller fp32 layers run on plain fp32 FMA kernels and need none. */
dp_status dp_ghost_norms(dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                         int32_t B, int32_t T, float* sq,
                         void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
size_t dp_ghost_norms_ws_bytes(const dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                               int32_t B, int32_t T);

/* ---- per-example norm of an embedding table's gradient (Eq. 4 with one-hot inputs) ----
 * ids [dev, (B,T) int32 in [0,V)]; G [dev, (B*T, d)] gradient reaching the embedding output;
 * first_occ [dev, (B,T) int32 or NULL]: smallest s with ids[i,s] == ids[i,t].
 * A learned position table is the same call with ids[i,t] = t and V = T.  T <= 4096. */
dp_status dp_embed_norms(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                         int32_t B, int32_t T, int32_t d, int32_t V, float* sq,
                         int32_t* first_occ, void* ws, size_t ws_bytes,
                         int32_t* dev_status, void* stream);
size_t dp_embed_norms_ws_bytes(int32_t B, int32_t T, int32_t d);

/* ---- the same embedding norm without any caller workspace ----
 * (No counterpart in the paper: this entry point exists for the way the library is hosted.)
 * For callers that cannot allocate or pass scratch memory -- code running while the host's
 * allocator is frozen for a step, plug-ins that receive only their input and output tensors,
 * devices whose memory is already fully committed.  The partial sums of the norm kernel live in
 * a fixed 64 KiB array inside the library image (every device that loads the library holds it
 * until the process exits), so B * ceil(d / 256) must not exceed DP_STATIC_SCRATCH_FLOATS,
 * else DP_ERR_SCRATCH_LIMIT is returned and nothing is enqueued.  Inputs, outputs and results
 * are those of dp_embed_norms.  No cudaMalloc / cudaFree or other allocating call is made.
 * The first call on each device looks up the array's device address (a host-side runtime
 * query); make that first call before starting any stream capture.  All calls on a device
 * share the one array: it keeps the previous call's contents (each call overwrites every
 * element it later reads, so nothing needs clearing), and two calls whose kernels may overlap
 * on the GPU -- different streams, no ordering between them -- race on it and must not be
 * issued. */
#define DP_STATIC_SCRATCH_FLOATS 16384
dp_status dp_embed_norms_static(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                int32_t B, int32_t T, int32_t d, int32_t V, float* sq,
                                int32_t* first_occ, int32_t* dev_status, void* stream);

/* ---- parameters that act element-wise along the feature axis: biases, LayerNorm ----
 * A bias sees the back-propagated signal of every token (Eq. 4 with a constant input 1): its
 * per-example gradient is v_i = sum_t G[i,t,:].  A LayerNorm gain has v_i = sum_t G[i,t,:] *
 * X[i,t,:], X the normalised input and G the gradient at the LayerNorm output; its shift is a
 * bias.  With these blocks Eq. 6 runs over every parameter of a GPT-2 model.
 * G, X [dev, (B*T, p)], X may be NULL (bias).  Any alignment works; 16-byte aligned tensors
 * with pitches that are multiples of 16 bytes take the vector-load path. */
typedef struct {
  const void* G;  int64_t ldg;
  const void* X;  int64_t ldx;      /* NULL / 0 for a bias */
  int32_t p;
} dp_vector_desc;
/* sq[i] += || v_i ||^2 for every parameter in params [host, n entries]. */
dp_status dp_vector_norms(const dp_vector_desc* params, int32_t n, dp_dtype dt, int32_t B,
                          int32_t T, float* sq, void* ws, size_t ws_bytes, void* stream);
size_t dp_vector_norms_ws_bytes(const dp_vector_desc* params, int32_t n, int32_t B, int32_t T);
/* outs[k] (p_k floats) = beta*outs[k] + sum_i R_i v_i, then, if with_noise, the Gaussian
 * mechanism outs[k] = scale * (outs[k] + sigma*C*z) with the stream (seed, tensor_ids[k], step)
 * of dp_add_noise.  outs, tensor_ids [host arrays, n entries; tensor_ids may be NULL without
 * noise].  clip [dev, B or NULL] receives R. */
dp_status dp_clip_accumulate_vectors(const dp_vector_desc* params, int32_t n, dp_dtype dt,
                                     int32_t B, int32_t T, const float* sq, float C, float* clip,
                                     float* const* outs, float beta, int32_t with_noise,
                                     float sigma, float scale, uint64_t seed,
                                     const uint32_t* tensor_ids, uint32_t step,
                                     void* ws, size_t ws_bytes, void* stream);
size_t dp_clip_accumulate_vectors_ws_bytes(const dp_vector_desc* params, int32_t n, int32_t B,
                                           int32_t T);

/* ---- cross term of a weight-tied embedding / LM head (Eq. 11, Eq. 13) ----
 * Adds 2*<g_in_i, g_out_i> to sq[i], with g_in_i the (V,d) embedding gradient of example i
 * and g_out_i = G_lm_i^T A_lm_i, through
 *    <g_in_i, g_out_i> = sum_{t,s} G_lm[i,s,ids[i,t]] * (G_emb[i,t,:] . A_lm[i,s,:])
 * so neither V x d matrix is formed.  cross [dev, B floats or NULL] receives the bare inner
 * product (overwritten).  G_emb, A_lm: (B*T, d); G_lm: (B*T, V). */
dp_status dp_tied_cross_term(const int32_t* ids, const void* G_emb, int64_t ldge,
                             const void* A_lm, int64_t ldal, const void* G_lm, int64_t ldgl,
                             dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t V,
                             float* sq, float* cross, void* ws, size_t ws_bytes,
                             int32_t* dev_status, void* stream);
size_t dp_tied_cross_term_ws_bytes(int32_t B, int32_t T, int32_t d, int32_t V);

/* ---- clip coefficients (Eq. 2, Eq. 7) ----
 * clip[i] = min(1, C / sqrt(sq[i])), 1 when sq[i] == 0 (no stabiliser is added);
 * norms [dev, B or NULL] receives sqrt(sq[i]).  C > 0 and finite.
 * Bad norms fail closed: a squared norm that is NaN or infinite gives clip[i] = 0 (the example
 * drops out of every clipped sum instead of entering it unclipped); a slightly negative one (the
 * tied sum in + out + 2 cross can round below zero when the true norm is ~0) counts as 0. */
dp_status dp_clip_factors(const float* sq, int32_t B, float C, float* clip, float* norms,
                          void* stream);
/* The same after joining a second accumulator: sq[i] += sq_extra[i] (one addition, fixed order),
 * then clip and norms from the sum.  For norm calls that ran on two streams into two
 * accumulators.  clip, norms [dev, B or NULL]. */
dp_status dp_clip_factors_sum(float* sq, const float* sq_extra, int32_t B, float C, float* clip,
                              float* norms, void* stream);
/* In every dp_clip_accumulate* call below, sq may be NULL: `clip` [dev, B] then is an INPUT that
 * already holds the factors R_i (from dp_clip_factors / dp_clip_factors_sum), and the call does
 * not recompute them -- one kernel less per call when a step makes several. */

/* ---- clipped sum of a linear layer: out = beta*out + sum_i R_i G_i^T A_i  (Eq. 3) ----
 * One GEMM with M = p, N = d, K = B*T whose K rows are scaled by R_i = min(1, C/sqrt(sq[i]))
 * on chip.  out [dev, (p,d) fp32, leading dimension ldo] has the layout of a linear layer's
 * weight gradient.  beta is 0 (overwrite) or 1 (accumulate).  clip [dev, B or NULL] receives
 * R.  This replaces the re-weighted second backward pass of ghost clipping by its result.
 * DP_F32 layers with T >= 32 and d, p >= 64 take the split-bf16 tensor-core path described at
 * dp_ghost_norms (R_i multiplies G in fp32 before the split); the workspace grows accordingly. */
dp_status dp_clip_accumulate(const void* A, int64_t lda, const void* G, int64_t ldg,
                             dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t p,
                             const float* sq, float C, float* clip,
                             float* out, int64_t ldo, float beta,
                             void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
size_t dp_clip_accumulate_ws_bytes(dp_dtype dt, int32_t B, int32_t T, int32_t d, int32_t p);

/* ---- the same clipped sums for many layers in ONE launch ----
 * layers [host, n_layers entries; mode fields ignored]; outs [host array of n_layers [dev]
 * pointers], ldos [host array].  The output tiles of all layers form one work list for a
 * persistent kernel, which keeps every SM busy even when a single layer has few tiles.
 * Same scalars, clip output and error rules as dp_clip_accumulate. */
dp_status dp_clip_accumulate_grouped(const dp_linear_desc* layers, int32_t n_layers, dp_dtype dt,
                                     int32_t B, int32_t T, const float* sq, float C, float* clip,
                                     float* const* outs, const int64_t* ldos, float beta,
                                     void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
size_t dp_clip_accumulate_grouped_ws_bytes(const dp_linear_desc* layers, int32_t n_layers,
                                           dp_dtype dt, int32_t B, int32_t T);

/* ---- clipped sum of an embedding table: out[v,:] = beta*out[v,:] + sum_{i,t: id=v} R_i g_{i,t} ----
 * The B*T token positions are ordered by a stable counting sort on the id, then every
 * distinct id is reduced in that order.  perm [dev, B*T int32 or NULL] and seg [dev, V+1
 * int32 or NULL] receive the sort: perm lists flat positions by (id, position) and
 * seg[v] = number of positions with id < v.  With a tied head, call with beta = 1 on the
 * matrix dp_clip_accumulate wrote for the head. */
dp_status dp_clip_accumulate_embed(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                   int32_t B, int32_t T, int32_t d, int32_t V,
                                   const float* sq, float C, float* clip,
                                   float* out, int64_t ldo, float beta,
                                   int32_t* perm, int32_t* seg,
                                   void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
size_t dp_clip_accumulate_embed_ws_bytes(int32_t B, int32_t T, int32_t d, int32_t V);

/* The same in two calls, so that the sort -- which needs only the ids -- can run early, e.g. on
 * a second stream while the norms are computed.  dp_embed_sort writes perm [dev, B*T int32] and
 * seg [dev, V+1 int32] as described above (ws of dp_embed_sort_ws_bytes);
 * dp_clip_accumulate_embed_sorted is dp_clip_accumulate_embed with that sort given (perm, seg
 * are inputs; ws of dp_clip_accumulate_embed_ws_bytes).  Out-of-range ids are flagged by the
 * sort (DP_DEV_BAD_ID) and skipped by both. */
dp_status dp_embed_sort(const int32_t* ids, int32_t B, int32_t T, int32_t V, int32_t* perm,
                        int32_t* seg, void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);
size_t dp_embed_sort_ws_bytes(int32_t B, int32_t T, int32_t V);
dp_status dp_clip_accumulate_embed_sorted(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                          int32_t B, int32_t T, int32_t d, int32_t V,
                                          const float* sq, float C, float* clip,
                                          float* out, int64_t ldo, float beta,
                                          const int32_t* perm, const int32_t* seg,
                                          void* ws, size_t ws_bytes, int32_t* dev_status, void* stream);

/* ---- clipped sums with the Gaussian mechanism fused in (Eq. 2, Eq. 3, Eq. 7 in one pass) ----
 * Same as dp_clip_accumulate_grouped, then outs[k] = scale * (outs[k] + sigma*C*z) with the
 * stream (seed, tensor_ids[k], step) of dp_add_noise, element j = row*d + col.  The noise is
 * generated in the GEMM epilogue, so the clipped sum is never re-read from memory.  Values are
 * identical to calling dp_clip_accumulate_grouped and then dp_add_noise on each tensor.
 * tensor_ids [host, n_layers].  Use the unfused calls when several devices must add their sums
 * before the single noise draw. */
dp_status dp_clip_accumulate_noise_grouped(const dp_linear_desc* layers, int32_t n_layers,
                                           dp_dtype dt, int32_t B, int32_t T, const float* sq,
                                           float C, float* clip, float* const* outs,
                                           const int64_t* ldos, float beta, float sigma, float scale,
                                           uint64_t seed, const uint32_t* tensor_ids, uint32_t step,
                                           void* ws, size_t ws_bytes, int32_t* dev_status,
                                           void* stream);
/* Embedding table with the Gaussian mechanism: beta == 0 fills the table with scale*sigma*C*z
 * (write only, in place of the zero fill) and adds scale * the clipped row sums; beta == 1 adds
 * scale * the clipped row sums to a table that already holds its noise (tied head).  Equal to the
 * unfused calls up to fp32 rounding order. */
dp_status dp_clip_accumulate_embed_noise(const int32_t* ids, const void* G, int64_t ldg, dp_dtype dt,
                                         int32_t B, int32_t T, int32_t d, int32_t V, const float* sq,
                                         float C, float* clip, float* out, int64_t ldo, float beta,
                                         float sigma, float scale, uint64_t seed, uint32_t tensor_id,
                                         uint32_t step, int32_t* perm, int32_t* seg, void* ws,
                                         size_t ws_bytes, int32_t* dev_status, void* stream);

/* ---- Gaussian mechanism: out[j] = scale * (out[j] + sigma*C*z_j)  (Eq. 3) ----
 * z_j is a pure function of (seed, tensor_id, step, j): Philox4x32-10 with key
 * (seed low word, seed high word) and counter (j/4 low, j/4 high, tensor_id, step); word
 * pairs (x0,x1), (x2,x3) go through Box-Muller with u1 = ((xa>>8)+1)/2^24,
 * u2 = (xb>>8)/2^24, giving r cos(2 pi u2) and r sin(2 pi u2) for elements 4q+{0,1} and
 * 4q+{2,3}.  out [dev, n floats, 16-byte aligned]; scale = 1 gives the noised sum,
 * scale = 1/|B| the full Eq. 3.  sigma >= 0, C > 0, all finite. */
dp_status dp_add_noise(float* out, int64_t n, float sigma, float C, float scale,
                       uint64_t seed, uint32_t tensor_id, uint32_t step, void* stream);

/* The same on a SLICE of a tensor: out [dev, n floats, 16-byte aligned] holds elements
 * first_element .. first_element+n-1 of the logical tensor and receives exactly the noise those
 * elements get from dp_add_noise on the whole tensor (first_element a multiple of 4, so that a
 * slice owns whole Philox counters; otherwise DP_ERR_ALIGNMENT).  For the data-parallel form in
 * which each rank owns a slice of the summed gradient after a reduce-scatter: the noise is drawn
 * once, on the owner, and equals the single-GPU stream. */
dp_status dp_add_noise_slice(float* out, int64_t n, int64_t first_element, float sigma, float C,
                             float scale, uint64_t seed, uint32_t tensor_id, uint32_t step,
                             void* stream);

/* Registers a device counter [dev, one uint32, must stay valid] whose current value is ADDED to
 * the `step` argument of every noise-drawing launch enqueued afterwards (NULL: none, the
 * default).  The kernels read it when they run, so a step captured once into a CUDA graph draws
 * fresh noise at each replay if the graph also increments the counter.  Process-wide setting;
 * not part of the paper (Eq. 3 only needs independent draws per step). */
dp_status dp_noise_step_device(const uint32_t* dev_counter);

/* Write-only form: out[j] = scale * sigma*C*z_j, the same stream as dp_add_noise on a zero
 * buffer.  It depends on no gradient, so it can run on a second stream while the norms are
 * computed; the clipped sums are then accumulated on top with beta = 1. */
dp_status dp_fill_noise(float* out, int64_t n, float sigma, float C, float scale,
                        uint64_t seed, uint32_t tensor_id, uint32_t step, void* stream);

/* ---- privacy accounting on the host (no device work) ----
 * The paper calibrates sigma with a Renyi-DP accountant from the target epsilon (3 in the main
 * experiments), delta = N^-1.1, the sampling rate q = batch / N and the number of steps.  One step
 * is the Poisson-subsampled Gaussian mechanism with sensitivity 1 (clipping to C, noise sigma*C);
 * for integer orders alpha = 2..256 its Renyi divergence is a binomial sum, RDP adds over steps,
 * and epsilon = min_alpha steps*rdp(alpha) + log(1/delta)/(alpha-1).
 * dp_rdp_epsilon: epsilon [host, out] and the minimising order best_order [host, out or NULL]
 * for 0 <= q <= 1, sigma > 0, steps >= 0, 0 < delta < 1 (else DP_ERR_INVALID_ARG).
 * dp_sigma_for_epsilon: the smallest sigma, to `tolerance`, whose epsilon does not exceed
 * target_epsilon (bisection; DP_ERR_UNSUPPORTED when the target is below what the conversion
 * term alone leaves).  All pointers are host pointers. */
dp_status dp_rdp_epsilon(double q, double sigma, int64_t steps, double delta, double* epsilon,
                         int32_t* best_order);
dp_status dp_sigma_for_epsilon(double q, int64_t steps, double target_epsilon, double delta,
                               double tolerance, double* sigma);

/* ---- helpers ---- */
const char* dp_status_string(dp_status s);
int32_t dp_last_cuda_error(void);      /* cudaError_t / CUresult of the last DP_ERR_CUDA */
const char* dp_version(void);
/* Number of CUDA kernels this library has enqueued since it was loaded (memsets and copies
 * are not counted).  Lets a caller report how many of its launches a timed region held. */
int64_t dp_kernel_launches(void);
/* Sets aside n SMs: every persistent kernel of the library (Gram, clipped-sum GEMM, cross term,
 * bias / LayerNorm passes) then sizes its grid for the device's SM count less n, so that kernels
 * of another stream -- the collectives of a data-parallel step, which cannot share an SM with
 * CTAs that take all of its shared memory -- find free SMs while a long launch is running instead
 * of waiting for its end.  Process-wide; applies to launches enqueued afterwards; the workspace
 * sizes depend on it, so set it before asking for them.  0 (the default) uses every SM; values are
 * clamped to [0, SMs - 2].  Returns the previous value.  Not part of the paper. */
int32_t dp_set_reserved_sms(int32_t n);
/* Test hook: when non-zero, linear-layer calls (DP_BF16 and DP_F32 alike) run the plain fp32-FMA
 * kernels instead of the tensor-core ones (used to cross-check the two on the device).  Returns
 * the previous value.  Off by default; not meant for production use. */
int32_t dp_debug_force_fma(int32_t on);
/* Test hook: when non-zero, sequences longer than 128 tokens keep the single-CTA 128 x 128 Gram
 * kernel instead of the CTA-pair 256 x 256 one (used to cross-check the two on the device).
 * Returns the previous value. */
int32_t dp_debug_ghost_single(int32_t on);
/* Diagnostics.  dp_debug_noise_error_scan: exhaustive float64 check of the fp32 Box-Muller
 * factors over all 2^24 inputs; out4 [dev, 4 doubles] = {max relative error of the radius for
 * r^2 <= t_max (t_max <= 0: the threshold in use), max absolute error of cos/sin, largest radius
 * seen, the compiled r^2 threshold}. */
dp_status dp_debug_noise_error_scan(float t_max, double* out4, void* stream);
/* The checked build (libdp_ghost_check.so, compiled with -DDP_BOUNDS_CHECK) compares every index
 * that a kernel computes from data with the extent of the array it addresses, ORs DP_DEV_BOUNDS
 * into dev_status for an index outside and skips that access: a stand-in for a memory checker.
 * dp_debug_bounds_checked: 1 in the checked build, 0 otherwise.  dp_debug_bounds_probe: runs the
 * range test on (idx, n) in a one-thread kernel that touches no memory, so that a test can see an
 * out-of-range index being reported without any invalid access.  dp_debug_tensor_map_encodes:
 * TMA tensor maps encoded by the driver so far (maps are cached per tensor and box shape). */
int32_t dp_debug_bounds_checked(void);
dp_status dp_debug_bounds_probe(int64_t idx, int64_t n, int32_t* dev_status, void* stream);
int64_t dp_debug_tensor_map_encodes(void);
/* Test knob for the failure path: device-side barrier waits give up after `cycles` (0: at the
 * first miss; negative: back to the default of about a second).  A kernel whose wait gives up
 * ORs DP_DEV_TIMEOUT into dev_status, lets its copies and MMAs in flight finish, frees its
 * tensor memory and returns; the context stays usable.  Returns the previous limit. */
int64_t dp_debug_set_wait_limit(int64_t cycles);

#ifdef __cplusplus
}
#endif
#endif /* DP_GHOST_H_ */
