// Cross term of a weight-tied embedding / LM head on tcgen05 tensor cores (Eq. 11, Eq. 13).
//
//   <g_in_i, g_out_i> = sum_{t,s} G_lm[i, s, id_t] * M_i[t, s],   M_i = G_emb_i A_lm_i^T  (T x T)
//
// with g_in_i the (V, d) embedding gradient and g_out_i = G_lm_i^T A_lm_i the head gradient of
// example i: neither V x d matrix is formed.  A work item is one 128 x 128 tile of M_i,
// accumulated in tensor memory over d (TMA-fed, K-major operands); the epilogue warps multiply
// every entry by the gathered logit gradient G_lm[i, s, id_t] and sum.  Partial sums go to a
// workspace and are added in a fixed order by the caller's reduce kernel.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "cross_term.cuh"
#include "dp_common.cuh"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace dpg {

namespace {

constexpr int kTile = 128;
constexpr int kKStep = 64;
constexpr int kTileBytes = kTile * kKStep * 2;       // 16 KiB
constexpr int kStageBytes = 2 * kTileBytes;          // G_emb row tile + A_lm row tile
constexpr int kStages = 6;
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;                       // 2 accumulators x 128 columns
constexpr size_t kSmemBytes = size_t(kStages) * kStageBytes + 1024 + 512;

struct __align__(64) CrossParams {
  CUtensorMap tmE;           // G_emb (B, T, d)
  CUtensorMap tmA;           // A_lm  (B, T, d)
  const int* ids;            // (B, T)
  const __nv_bfloat16* Glm;  // (B*T, V) logit gradients
  long long ldgl;
  int B, T, V, nt, ksteps;
  int total_items;           // B * nt * nt
  float* partials;           // [B][nt*nt]
  int* dev_status;
  long long wait_limit;
};

__global__ void __launch_bounds__(kThreads, 1)
cross_term_tc_kernel(const __grid_constant__ CrossParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + size_t(kStages) * kStageBytes);
  uint64_t* full = bars;
  uint64_t* empty = bars + kStages;
  uint64_t* acc_full = bars + 2 * kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* mma_done = acc_empty + 2;
  uint64_t* red_bar = mma_done + 1;                           // [4] epilogue warps -> warp 0
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(red_bar + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* epi_red = reinterpret_cast<float*>(tmem_slot + 2);   // [4][4]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { ptx::mbar_init(&acc_full[b], 1); ptx::mbar_init(&acc_empty[b], 4); }
    ptx::mbar_init(mma_done, 1);
    for (int b = 0; b < 4; ++b) ptx::mbar_init(&red_bar[b], 4);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) { ptx::tmem_alloc(tmem_slot, kTmemCols); ptx::tmem_relinquish(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int per_ex = P.nt * P.nt;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x) {
        const int ex = item / per_ex, tp = item % per_ex, ti = tp / P.nt, tj = tp % P.nt;
        for (int k = 0; k < P.ksteps; ++k) {
          if (!ptx::mbar_wait(&empty[stage], phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
          uint8_t* dst = tiles + size_t(stage) * kStageBytes;
          ptx::mbar_arrive_expect_tx(&full[stage], kStageBytes);
          ptx::tma_load_3d(dst, &P.tmE, &full[stage], k * kKStep, ti * kTile, ex);
          ptx::tma_load_3d(dst + kTileBytes, &P.tmA, &full[stage], k * kKStep, tj * kTile, ex);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_copies(full, kStages, issued);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTile, kTile, 0, 0);
      constexpr uint64_t dbase = ptx::smem_desc_base(16, 1024, ptx::SWIZZLE_128B);
      uint32_t stage = 0, phase = 0, n_item = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x, ++n_item) {
        const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
        if (!ptx::mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kTile;
        for (int k = 0; k < P.ksteps; ++k) {
          if (!ptx::mbar_wait(&full[stage], phase, abort_flag, P.wait_limit)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t se = ptx::smem_u32(tiles + size_t(stage) * kStageBytes);
          const uint32_t sa = se + kTileBytes;
#pragma unroll
          for (int kk = 0; kk < kKStep / 16; ++kk)
            ptx::mma_bf16_ss(d_tmem, ptx::smem_desc(dbase, se + kk * 32),
                             ptx::smem_desc(dbase, sa + kk * 32), idesc, (k > 0 || kk > 0) ? 1u : 0u);
          ptx::mma_commit(&empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) ptx::mma_commit(&acc_full[buf]);
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_mmas(mma_done, false);
      }
    }
  } else {
    const int q = warp & 3, ew = warp - 2;
    uint32_t n_item = 0;
    bool ok = true;
    for (int item = blockIdx.x; item < P.total_items && ok; item += gridDim.x, ++n_item) {
      const int ex = item / per_ex, tp = item % per_ex, ti = tp / P.nt, tj = tp % P.nt;
      const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
      // this thread's token t and the column of G_lm it gathers from
      const int t = ti * kTile + q * 32 + lane;
      int id = -1;
      if (t < P.T) {
        id = P.ids[size_t(ex) * P.T + t];
        if (id < 0 || id >= P.V) {
          if (P.dev_status) atomicOr(P.dev_status, DP_DEV_BAD_ID);
          id = -1;                                   // skipped token
        }
      }
      const __nv_bfloat16* gcol = P.Glm + size_t(ex) * P.T * P.ldgl + (id >= 0 ? id : 0);
      if (!ptx::mbar_wait_relaxed(&acc_full[buf], acc_phase, abort_flag, P.wait_limit)) { ok = false; break; }
      ptx::tc_fence_after();
      const uint32_t t0 = tmem_base + (uint32_t(q * 32) << 16) + buf * kTile;
      float acc = 0.f;
#pragma unroll 1
      for (int c = 0; c < kTile / 32; ++c) {
        uint32_t r[32];
        ptx::tmem_ld_32x32b_x32(t0 + c * 32, r);
        ptx::tmem_ld_wait();
        const int s0 = tj * kTile + c * 32;
        float wv[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          // gathered logit gradient G_lm[ex, s0 + j, id]: the flat element index is computed from
          // the token id, so the checked build compares it with the tensor's extent
          const bool take = id >= 0 && s0 + j < P.T &&
                            dp_in_range((long long)(size_t(ex) * P.T + s0 + j) * P.ldgl + id,
                                        (long long)P.B * P.T * P.ldgl, P.dev_status);
          wv[j] = take ? __bfloat162float(gcol[size_t(s0 + j) * P.ldgl]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) acc = fmaf(__uint_as_float(r[j]), wv[j], acc);
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
      // the four warps' sums meet through an mbarrier with a bounded wait (no blocking named
      // barrier: a warp that gave up never arrives); four slots, since the other warps can run at
      // most two items ahead of a waiting warp 0
      acc = warp_sum(acc);
      const uint32_t slot = n_item & 3, red_phase = (n_item >> 2) & 1;
      if (lane == 0) { epi_red[slot * 4 + ew] = acc; ptx::mbar_arrive(&red_bar[slot]); }
      if (ew == 0) {
        if (!ptx::mbar_wait_relaxed(&red_bar[slot], red_phase, abort_flag, P.wait_limit)) { ok = false; break; }
        if (lane == 0 && dp_in_range(item, P.total_items, P.dev_status))
          P.partials[item] = (epi_red[slot * 4 + 0] + epi_red[slot * 4 + 1]) +
                             (epi_red[slot * 4 + 2] + epi_red[slot * 4 + 3]);
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

}  // namespace

int cross_term_tc_partials_per_example(int T) {
  const int nt = ceil_div(T, kTile);
  return nt * nt;
}

dp_status launch_cross_term_tc(const int* ids, const void* Ge, int64_t ldge, const void* Al,
                               int64_t ldal, const void* Gl, int64_t ldgl, int B, int T, int d, int V,
                               float* partials, int* dev_status, cudaStream_t st) {
  if (first_use_on_this_device(reinterpret_cast<const void*>(&cross_term_tc_kernel)))
    DP_CUDA_OK(cudaFuncSetAttribute(cross_term_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kSmemBytes));
  CrossParams P;
  memset(&P, 0, sizeof(P));
  dp_status s = make_tmap_bf16_3d(&P.tmE, Ge, ldge, d, T, B, kKStep, kTile);
  if (s != DP_OK) return s;
  s = make_tmap_bf16_3d(&P.tmA, Al, ldal, d, T, B, kKStep, kTile);
  if (s != DP_OK) return s;
  P.ids = ids;
  P.Glm = static_cast<const __nv_bfloat16*>(Gl);
  P.ldgl = ldgl;
  P.B = B; P.T = T; P.V = V;
  P.nt = ceil_div(T, kTile);
  P.ksteps = ceil_div(d, kKStep);
  P.total_items = B * P.nt * P.nt;
  P.partials = partials;
  P.dev_status = dev_status;
  P.wait_limit = g_wait_limit;
  const int grid = std::min(P.total_items, sm_count());
  cross_term_tc_kernel<<<grid, kThreads, kSmemBytes, st>>>(P);
  DP_LAUNCH_OK();
  return DP_OK;
}

}  // namespace dpg
