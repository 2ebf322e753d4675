// Ghost norm of linear layers on tcgen05 tensor cores (bf16 in, fp32 accumulate).
//
// For example i and a linear layer with input A_i (T x d) and output gradient G_i (T x p),
// the squared Frobenius norm of the per-example weight gradient G_i^T A_i equals
// <A_i A_i^T, G_i G_i^T>_F (Eq. 4 - Eq. 5 extended from one token to T tokens).  A work item
// is one 128 x 128 tile pair (ti <= tj) of the two T x T Gram matrices of one (layer,
// example): both tiles are accumulated in tensor memory, multiplied element by element and
// summed by the epilogue warps; off-diagonal tile pairs count twice (symmetry).
//
// The Frobenius product is linear in each Gram matrix, so a very wide operand (the LM head's
// V = 50257 columns) is split into column chunks handled by different CTAs; each chunk CTA
// recomputes the full Gram tile of the narrow operand.
//
// Roles per CTA (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (one thread),
// warps 2..5 = epilogue.  Two TMEM accumulator sets let the epilogue of one item overlap the
// MMAs of the next.  Partial sums go to a workspace and are added in a fixed order by a
// second kernel, so results are deterministic.
#include <cuda.h>
#include <cuda_bf16.h>

#include "dp_common.cuh"
#include "ghost_plan.cuh"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace dpg {

namespace {

constexpr int kTile = 128;                       // Gram tile edge (rows of A_i / G_i)
constexpr int kKStep = 64;                       // bf16 columns per stage row (128 bytes)
constexpr int kTileBytes = kTile * kKStep * 2;   // 16 KiB
// A stage holds row tile ti and, for off-diagonal tile pairs, row tile tj.  When T <= 128 every
// pair is diagonal, so stages shrink to one tile and twice as many are kept in flight (the
// kernel is HBM-bound there: bytes in flight are what counts).
template <bool kDiagOnly>
struct GhostGeo {
  static constexpr int kStageBytes = kDiagOnly ? kTileBytes : 2 * kTileBytes;
  static constexpr int kStages = kDiagOnly ? 12 : 6;
  static constexpr size_t kSmemBytes = size_t(kStages) * kStageBytes + 1024 /*alignment slack*/ + 512;
};
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;                   // 2 buffers x (S_A 128 + S_G 128) columns

struct __align__(64) GhostParams {
  CUtensorMap tmA[kGhostMaxLayers];
  CUtensorMap tmG[kGhostMaxLayers];
  GhostLayerPlan layer[kGhostMaxLayers];
  int n_layers;
  int B, T, nt, ntp;
  int total_items;
  int n_per;                 // partial sums per example in the workspace
  float* partials;           // [B][n_per]
  int* dev_status;
  long long wait_limit;      // cycles a barrier wait may take before the CTA gives up
};

struct Item {
  int layer, example, ti, tj, a0, a1, g0, g1, pidx;
};

__device__ __forceinline__ Item decode_item(const GhostParams& P, int item) {
  Item it;
  int l = 0;
  while (l + 1 < P.n_layers && item >= P.layer[l + 1].item_begin) ++l;
  const GhostLayerPlan& L = P.layer[l];
  const int local = item - L.item_begin;
  const int s = local % L.nsplit;
  const int tp = (local / L.nsplit) % P.ntp;
  it.example = local / (L.nsplit * P.ntp);
  it.layer = l;
  int ti = 0, rem = tp;                   // tile pairs enumerated row by row, tj >= ti
  while (rem >= P.nt - ti) { rem -= P.nt - ti; ++ti; }
  it.ti = ti;
  it.tj = ti + rem;
  const int c0 = s * L.chunk_steps;
  if (L.split_on_g) {
    it.a0 = 0; it.a1 = L.a_steps;
    it.g0 = c0; it.g1 = min(c0 + L.chunk_steps, L.g_steps);
  } else {
    it.g0 = 0; it.g1 = L.g_steps;
    it.a0 = c0; it.a1 = min(c0 + L.chunk_steps, L.a_steps);
  }
  it.pidx = it.example * P.n_per + L.col_begin + tp * L.nsplit + s;
  return it;
}

// kDual: the two sides of each Gram product come from two different tensors (maps 2l and 2l+1 of
// a layer): the fp32 path, where S = X Y^T with X = [hi | hi | lo] and Y = [hi | lo | hi] of the
// operand split into two bf16 terms.  S is still symmetric, so tile pairs are enumerated as before,
// but a diagonal pair also needs both loads.
template <bool kDiagOnly, bool kDual = false>
__global__ void __launch_bounds__(kThreads, 1)
ghost_norm_tc_kernel(const __grid_constant__ GhostParams P) {
  static_assert(!(kDiagOnly && kDual), "the two-tensor form always loads two tiles per stage");
  constexpr int kStages = GhostGeo<kDiagOnly>::kStages;
  constexpr int kStageBytes = GhostGeo<kDiagOnly>::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  // 128-byte swizzled tiles need 1024-byte alignment
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + size_t(kStages) * kStageBytes);
  uint64_t* full = bars;                   // [kStages]  TMA -> MMA
  uint64_t* empty = bars + kStages;        // [kStages]  MMA -> TMA
  uint64_t* acc_full = bars + 2 * kStages; // [2]        MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;      // [2]        epilogue -> MMA
  uint64_t* mma_done = acc_empty + 2;      // only used when the MMA issuer gives up
  uint64_t* red_bar = mma_done + 1;        // [4]        epilogue warps -> epilogue warp 0
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(red_bar + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* epi_red = reinterpret_cast<float*>(tmem_slot + 2);   // [4][4]

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 4); }
    ptx::mbar_init(mma_done, 1);
    for (int b = 0; b < 4; ++b) ptx::mbar_init(&red_bar[b], 4);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {                    // one warp owns the TMEM allocation
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x) {
        const Item it = decode_item(P, item);
        const bool diag = !kDual && (kDiagOnly || (it.ti == it.tj));
        const uint32_t bytes = diag ? kTileBytes : kStageBytes;
        const int li = kDual ? 2 * it.layer : it.layer;
        for (int pass = 0; pass < 2 && ok; ++pass) {
          const CUtensorMap* tm = pass == 0 ? &P.tmA[li] : &P.tmG[li];
          const CUtensorMap* tm2 = kDual ? tm + 1 : tm;     // the other side of the product
          const int k0 = pass == 0 ? it.a0 : it.g0, k1 = pass == 0 ? it.a1 : it.g1;
          for (int k = k0; k < k1; ++k) {
            if (!ptx::mbar_wait(&empty[stage], phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
            uint8_t* dst = tiles + size_t(stage) * kStageBytes;
            ptx::mbar_arrive_expect_tx(&full[stage], bytes);
            ptx::tma_load_3d(dst, tm, &full[stage], k * kKStep, it.ti * kTile, it.example);
            if (!diag)
              ptx::tma_load_3d(dst + kTileBytes, tm2, &full[stage], k * kKStep, it.tj * kTile,
                               it.example);
            ++issued;
            if (++stage == kStages) { stage = 0; phase ^= 1; }
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_copies(full, kStages, issued);   // copies in flight land before exit
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);
      // K-major operand, 128-byte swizzle: 8-row groups are 1024 bytes apart
      constexpr uint64_t dbase = ptx::smem_desc_base(16, 1024, ptx::SWIZZLE_128B);
      uint32_t stage = 0, phase = 0, n_item = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x, ++n_item) {
        const Item it = decode_item(P, item);
        const bool diag = !kDual && (kDiagOnly || (it.ti == it.tj));
        const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
        if (!ptx::mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
        ptx::tc_fence_after();
        for (int pass = 0; pass < 2 && ok; ++pass) {
          const uint32_t d_tmem = tmem_base + buf * 256 + pass * 128;
          const int nsteps = pass == 0 ? it.a1 - it.a0 : it.g1 - it.g0;
          for (int k = 0; k < nsteps; ++k) {
            if (!ptx::mbar_wait(&full[stage], phase, abort_flag, P.wait_limit)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t sa = ptx::smem_u32(tiles + size_t(stage) * kStageBytes);
            const uint32_t sb = diag ? sa : sa + kTileBytes;
#pragma unroll
            for (int kk = 0; kk < kKStep / 16; ++kk) {
              // 16 bf16 = 32 bytes further along K inside the swizzle atom
              ptx::mma_bf16_ss(d_tmem, ptx::smem_desc(dbase, sa + kk * 32),
                               ptx::smem_desc(dbase, sb + kk * 32), idesc,
                               (k > 0 || kk > 0) ? 1u : 0u);
            }
            ptx::mma_commit(&empty[stage]);          // stage reusable once these MMAs retire
            if (++stage == kStages) { stage = 0; phase ^= 1; }
          }
        }
        if (ok) ptx::mma_commit(&acc_full[buf]);     // both Gram tiles complete
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_mmas(mma_done, false);
      }
    }
  } else {
    // ----------------------------------------------------------------- epilogue
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int ew = warp - 2;
    uint32_t n_item = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x, ++n_item) {
      const Item it = decode_item(P, item);
      const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
      if (!ptx::mbar_wait_relaxed(&acc_full[buf], acc_phase, abort_flag, P.wait_limit)) { ok = false; break; }
      ptx::tc_fence_after();
      const uint32_t t0 = tmem_base + (uint32_t(q * 32) << 16) + buf * 256;
      float acc = 0.f;
#pragma unroll 1
      for (int c = 0; c < kTile / 32; ++c) {
        uint32_t ra[32], rg[32];
        ptx::tmem_ld_32x32b_x32(t0 + c * 32, ra);
        ptx::tmem_ld_32x32b_x32(t0 + 128 + c * 32, rg);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) acc = fmaf(__uint_as_float(ra[j]), __uint_as_float(rg[j]), acc);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);   // accumulators may be overwritten
      // The four warps' sums meet through an mbarrier, not a blocking named barrier: a warp that
      // gave up above never arrives, and warp 0's wait for the others is bounded like every other.
      // Four slots: the other warps can run at most two items ahead of a waiting warp 0 (they
      // need its acc_empty arrivals), so a slot is never rewritten before it has been read.
      acc = warp_sum(acc);
      const uint32_t slot = n_item & 3, red_phase = (n_item >> 2) & 1;
      if (lane == 0) { epi_red[slot * 4 + ew] = acc; ptx::mbar_arrive(&red_bar[slot]); }
      if (ew == 0) {
        if (!ptx::mbar_wait_relaxed(&red_bar[slot], red_phase, abort_flag, P.wait_limit)) { ok = false; break; }
        if (lane == 0 && dp_in_range(it.pidx, (long long)P.B * P.n_per, P.dev_status)) {
          const float s = (epi_red[slot * 4 + 0] + epi_red[slot * 4 + 1]) +
                          (epi_red[slot * 4 + 2] + epi_red[slot * 4 + 3]);
          P.partials[it.pidx] = (it.ti == it.tj) ? s : 2.f * s;
        }
      }
    }
    if (!ok && lane == 0) {
      *abort_flag = 1;
      if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

__global__ void reduce_partials_kernel(const float* __restrict__ partials, int n_per, int B,
                                       float* __restrict__ sq, float factor,
                                       float* __restrict__ plain_out) {
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (i >= B) return;
  float s = 0.f;
  for (int j = lane; j < n_per; j += 32) s += partials[size_t(i) * n_per + j];
  s = warp_sum(s);
  if (lane == 0) {
    if (plain_out) plain_out[i] = s;
    if (sq) sq[i] += factor * s;
  }
}

}  // namespace

dp_status launch_reduce_partials(const float* partials, int n_per, int B, float* sq,
                                 float factor, float* plain_out, cudaStream_t st) {
  const int warps = 4;
  reduce_partials_kernel<<<ceil_div(B, warps), warps * 32, 0, st>>>(partials, n_per, B, sq,
                                                                  factor, plain_out);
  DP_LAUNCH_OK();
  return DP_OK;
}

// Enqueue the tensor-core ghost norm for the planned layers; partial sums land in
// plan.partials layout inside `partials` (the caller reduces them afterwards).
dp_status launch_ghost_norm_tc(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                               float* partials, int* dev_status, cudaStream_t st,
                               const dp_linear_desc* other_side) {
  if (first_use_on_this_device(reinterpret_cast<const void*>(&launch_ghost_norm_tc))) {
    DP_CUDA_OK(cudaFuncSetAttribute(ghost_norm_tc_kernel<true>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)GhostGeo<true>::kSmemBytes));
    DP_CUDA_OK(cudaFuncSetAttribute(ghost_norm_tc_kernel<false>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)GhostGeo<false>::kSmemBytes));
    DP_CUDA_OK(cudaFuncSetAttribute(ghost_norm_tc_kernel<false, true>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)GhostGeo<false>::kSmemBytes));
  }
  const bool dual = other_side != nullptr;
  const size_t per_launch = dual ? kGhostMaxLayers / 2 : kGhostMaxLayers;
  const int nt = ceil_div(T, kTile);
  // layers are processed in groups that fit one parameter block
  for (size_t g0 = 0; g0 < plan.ghost_layers.size(); g0 += per_launch) {
    const size_t g1 = std::min(plan.ghost_layers.size(), g0 + per_launch);
    GhostParams P;
    memset(&P, 0, sizeof(P));
    int items = 0;
    for (size_t g = g0; g < g1; ++g) {
      const int li = plan.ghost_layers[g];
      const dp_linear_desc& L = layers[li];
      const size_t slot = dual ? 2 * (g - g0) : (g - g0);
      dp_status s = make_tmap_bf16_3d(&P.tmA[slot], L.A, L.lda, L.d, T, B, kKStep, kTile);
      if (s != DP_OK) return s;
      s = make_tmap_bf16_3d(&P.tmG[slot], L.G, L.ldg, L.p, T, B, kKStep, kTile);
      if (s != DP_OK) return s;
      if (dual) {
        const dp_linear_desc& R = other_side[li];
        s = make_tmap_bf16_3d(&P.tmA[slot + 1], R.A, R.lda, R.d, T, B, kKStep, kTile);
        if (s != DP_OK) return s;
        s = make_tmap_bf16_3d(&P.tmG[slot + 1], R.G, R.ldg, R.p, T, B, kKStep, kTile);
        if (s != DP_OK) return s;
      }
      GhostLayerPlan lp = plan.layer[li];
      lp.item_begin = items;
      items += B * plan.ntp * lp.nsplit;
      P.layer[g - g0] = lp;
    }
    P.n_layers = int(g1 - g0);
    P.B = B; P.T = T; P.nt = nt; P.ntp = plan.ntp;
    P.total_items = items;
    P.n_per = plan.n_per;
    P.partials = partials;
    P.dev_status = dev_status;
    P.wait_limit = g_wait_limit;
    const int grid = std::min(items, sm_count());
    if (dual)
      ghost_norm_tc_kernel<false, true><<<grid, kThreads, GhostGeo<false>::kSmemBytes, st>>>(P);
    else if (nt == 1)
      ghost_norm_tc_kernel<true><<<grid, kThreads, GhostGeo<true>::kSmemBytes, st>>>(P);
    else
      ghost_norm_tc_kernel<false><<<grid, kThreads, GhostGeo<false>::kSmemBytes, st>>>(P);
    DP_LAUNCH_OK();
  }
  return DP_OK;
}

}  // namespace dpg
