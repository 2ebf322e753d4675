// Ghost norm of linear layers for sequences longer than 128 tokens, on CTA pairs.
//
// Same quantity as ghost_norm_tc.cu -- <A_i A_i^T, G_i G_i^T>_F per example and layer (Eq. 4 -
// Eq. 5 extended from one token to T tokens) -- but a work item is one 256 x 256 tile pair
// (I <= J) of the two T x T Gram matrices, computed by two CTAs with cta_group::2 MMAs: each CTA
// loads 128 rows of row block I and 128 rows of row block J per 64-column K step (32 KiB for
// 2 x 128 x 256 x 64 multiply-adds), half the shared-memory fill per flop of a 128 x 128 tile.
// With T > 128 the single-CTA kernel is bound by the L2 -> SM fill rate, not by the tensor pipe;
// the larger tile trades 20 - 33 % more flops (the diagonal 256 x 256 tiles are computed in full)
// for half the operand traffic.
//
// Tensor memory holds S_A in columns 0..255 and S_G in columns 256..511 of each CTA (its 128 rows
// of the tile).  There is no room for a second pair of accumulators, so the overlap is in time:
// the epilogue warps copy S_A into registers while the MMAs of S_G run, which frees S_A for the
// next item before S_G is complete, and they multiply S_G against those registers while the next
// item's S_A is being accumulated.
//
// Roles per CTA (640 threads): warp 0 TMA producer, warp 1 MMA issuer (rank 0 only), warp 2 tells
// rank 0 that this CTA's half of a stage has landed, warp 3 idle, warps 4..19 epilogue (four per
// TMEM lane quarter, 64 columns each).  Every wait is bounded.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "dp_common.cuh"
#include "ghost_plan.cuh"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace dpg {

namespace {

constexpr int kRows = 128;                        // rows of a block that one CTA supplies
constexpr int kTile2 = 2 * kRows;                 // Gram tile edge of the pair
constexpr int kKStep = 64;                        // bf16 columns per stage row (128 bytes)
constexpr int kTileBytes = kRows * kKStep * 2;    // 16 KiB
constexpr int kStageBytes = 2 * kTileBytes;       // rows of block I, rows of block J
constexpr int kStages = 7;
constexpr size_t kSmemBytes = size_t(kStages) * kStageBytes + 1024 /*alignment slack*/ + 1024;
constexpr int kEpiWarp0 = 4, kEpiWarps = 16;
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;
constexpr int kColsPerWarp = kTile2 / (kEpiWarps / 4);    // 64

struct __align__(64) PairParams {
  CUtensorMap tmA[kGhostMaxLayers];
  CUtensorMap tmG[kGhostMaxLayers];
  GhostLayerPlan layer[kGhostMaxLayers];
  int n_layers;
  int B, T, nt, ntp;         // nt = ceil(T / 256) row blocks, ntp = nt (nt + 1) / 2 tile pairs
  int total_items;
  int n_per;
  float* partials;           // [B][n_per]; an item owns two consecutive slots (one per CTA)
  int* dev_status;
  long long wait_limit;
};
static_assert(sizeof(PairParams) <= 32000, "kernel parameter block too large");

struct Item {
  int layer, example, ti, tj, a0, a1, g0, g1, pidx;
};

__device__ __forceinline__ Item decode_item(const PairParams& P, int item) {
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
  it.pidx = it.example * P.n_per + L.col_begin + (tp * L.nsplit + s) * 2;
  return it;
}

__global__ void __launch_bounds__(kThreads, 1)
ghost_norm_pair_kernel(const __grid_constant__ PairParams P) {
  const uint32_t rank = ptx::cluster_ctarank();
  const int first_item = int(blockIdx.x >> 1);
  const int item_stride = int(gridDim.x >> 1);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + size_t(kStages) * kStageBytes);
  uint64_t* full = bars;                       // [kStages] this CTA's TMA landed
  uint64_t* ready = bars + kStages;            // [kStages] both CTAs' tiles landed (rank 0's copy)
  uint64_t* empty = bars + 2 * kStages;        // [kStages] MMAs retired
  uint64_t* sa_full = bars + 3 * kStages;      // S_A complete
  uint64_t* sg_full = sa_full + 1;             // S_G complete
  uint64_t* sa_empty = sa_full + 2;            // S_A copied to registers in both CTAs (rank 0's copy)
  uint64_t* sg_empty = sa_full + 3;            // S_G consumed in both CTAs (rank 0's copy)
  uint64_t* mma_done = sa_full + 4;
  uint64_t* red_bar = mma_done + 1;            // [4] this CTA's epilogue warps -> its epilogue warp 0
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(red_bar + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* epi_red = reinterpret_cast<float*>(tmem_slot + 2);   // [4][kEpiWarps]
  uint32_t* sink = reinterpret_cast<uint32_t*>(epi_red + 4 * kEpiWarps);   // [kStages] written by st.async, never read

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&ready[s], 1);             // rank 0's relay arrives and announces 4 bytes, rank 1's sends them
      ptx::mbar_init(&empty[s], 1);
    }
    ptx::mbar_init(sa_full, 1);
    ptx::mbar_init(sg_full, 1);
    ptx::mbar_init(sa_empty, kEpiWarps * 2);
    ptx::mbar_init(sg_empty, kEpiWarps * 2);
    ptx::mbar_init(mma_done, 1);
    for (int b = 0; b < 4; ++b) ptx::mbar_init(&red_bar[b], kEpiWarps);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) { ptx::tmem_alloc_pair(tmem_slot, kTmemCols); ptx::tmem_relinquish_pair(); }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_sync_all();        // the partner's barriers exist before anyone arrives on them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride) {
        const Item it = decode_item(P, item);
        const bool diag = it.ti == it.tj;
        const uint32_t bytes = diag ? kTileBytes : kStageBytes;
        const int row_i = it.ti * kTile2 + int(rank) * kRows;     // this CTA's rows of block I
        const int row_j = it.tj * kTile2 + int(rank) * kRows;     // and of block J
        for (int pass = 0; pass < 2 && ok; ++pass) {
          const CUtensorMap* tm = pass == 0 ? &P.tmA[it.layer] : &P.tmG[it.layer];
          const int k0 = pass == 0 ? it.a0 : it.g0, k1 = pass == 0 ? it.a1 : it.g1;
          for (int k = k0; k < k1; ++k) {
            if (!ptx::mbar_wait(&empty[stage], phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
            uint8_t* dst = tiles + size_t(stage) * kStageBytes;
            ptx::mbar_arrive_expect_tx(&full[stage], bytes);
            ptx::tma_load_3d(dst, tm, &full[stage], k * kKStep, row_i, it.example);
            if (!diag) ptx::tma_load_3d(dst + kTileBytes, tm, &full[stage], k * kKStep, row_j, it.example);
            ++issued;
            if (++stage == kStages) { stage = 0; phase ^= 1; }
          }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_copies(full, kStages, issued);
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------------- MMA issuer
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTile2, kTile2, 0, 0);
      constexpr uint64_t dbase = ptx::smem_desc_base(16, 1024, ptx::SWIZZLE_128B);   // K-major
      uint32_t stage = 0, phase = 0, n_item = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride, ++n_item) {
        const Item it = decode_item(P, item);
        const bool diag = it.ti == it.tj;
        const uint32_t ph = n_item & 1;
        for (int pass = 0; pass < 2 && ok; ++pass) {
          // the accumulator of this pass must have been read out for the previous item
          uint64_t* freed = pass == 0 ? sa_empty : sg_empty;
          if (!ptx::mbar_wait_cluster(freed, ph ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t d_tmem = tmem_base + pass * kTile2;
          const int nsteps = pass == 0 ? it.a1 - it.a0 : it.g1 - it.g0;
          for (int k = 0; k < nsteps; ++k) {
            if (!ptx::mbar_wait_cluster(&ready[stage], phase, abort_flag, P.wait_limit)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint32_t sa = ptx::smem_u32(tiles + size_t(stage) * kStageBytes);
            const uint32_t sb = diag ? sa : sa + kTileBytes;
#pragma unroll
            for (int kk = 0; kk < kKStep / 16; ++kk)
              ptx::mma_bf16_ss_pair(d_tmem, ptx::smem_desc(dbase, sa + kk * 32),
                                    ptx::smem_desc(dbase, sb + kk * 32), idesc,
                                    (k > 0 || kk > 0) ? 1u : 0u);
            ptx::mma_commit_pair(&empty[stage], 3);
            if (++stage == kStages) { stage = 0; phase ^= 1; }
          }
          if (ok) ptx::mma_commit_pair(pass == 0 ? sa_full : sg_full, 3);
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_mmas(mma_done, true);
      }
    }
  } else if (warp == 2) {
    // -------------------------------------------------------------------- relay
    // Tells rank 0's MMA issuer that this CTA's half of a stage has landed.  Rank 0's relay
    // arrives on its own `ready` barrier and announces 4 more bytes; rank 1's relay, which has
    // acquired its `full` barrier (so the TMA data are visible to it), delivers those 4 bytes with
    // an asynchronous store into rank 0's shared memory whose completion on the barrier is a
    // release at cluster scope.
    if (lane == 0) {
      const uint32_t ready_a = ptx::smem_u32(ready), sink_a = ptx::smem_u32(sink);
      const uint32_t ready_remote = ptx::mapa_u32(ready_a, 0), sink_remote = ptx::mapa_u32(sink_a, 0);
      uint32_t stage = 0, phase = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride) {
        const Item it = decode_item(P, item);
        const int nsteps = (it.a1 - it.a0) + (it.g1 - it.g0);
        for (int k = 0; k < nsteps; ++k) {
          if (!ptx::mbar_wait(&full[stage], phase, abort_flag, P.wait_limit)) { ok = false; break; }
          if (rank == 0) ptx::mbar_arrive_expect_tx_a(ready_a + 8 * stage, 4);
          else ptx::st_async_signal_a(ready_remote + 8 * stage, sink_remote + 4 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ----------------------------------------------------------------- epilogue
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int ew = warp - kEpiWarp0;
    const int cg = ew >> 2;                          // which 64 of the 256 columns
    const uint32_t t_sa = tmem_base + (uint32_t(q * 32) << 16) + cg * kColsPerWarp;
    const uint32_t t_sg = t_sa + kTile2;
    uint32_t n_item = 0;
    bool ok = true;
    for (int item = first_item; item < P.total_items && ok; item += item_stride, ++n_item) {
      const Item it = decode_item(P, item);
      const uint32_t ph = n_item & 1;
      // S_A -> registers, then the accumulator is free for the next item
      if (!ptx::mbar_wait_relaxed(sa_full, ph, abort_flag, P.wait_limit)) { ok = false; break; }
      ptx::tc_fence_after();
      uint32_t sa0[32], sa1[32];
      ptx::tmem_ld_32x32b_x32(t_sa, sa0);
      ptx::tmem_ld_32x32b_x32(t_sa + 32, sa1);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(sa_empty, 0);
      // S_G against the registers
      if (!ptx::mbar_wait_relaxed(sg_full, ph, abort_flag, P.wait_limit)) { ok = false; break; }
      ptx::tc_fence_after();
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t g[16];
        ptx::tmem_ld_32x32b_x16(t_sg + c * 16, g);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t a = (c < 2) ? sa0[(c & 1) * 16 + j] : sa1[(c & 1) * 16 + j];
          acc = fmaf(__uint_as_float(a), __uint_as_float(g[j]), acc);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_cluster(sg_empty, 0);
      // the warps' sums meet through an mbarrier with a bounded wait (no blocking named barrier:
      // a warp that gave up never arrives); four slots, since the other warps can run at most one
      // item ahead of a waiting warp 0 (they need its sa_empty arrival)
      acc = warp_sum(acc);
      const uint32_t slot = n_item & 3, red_phase = (n_item >> 2) & 1;
      if (lane == 0) { epi_red[slot * kEpiWarps + ew] = acc; ptx::mbar_arrive(&red_bar[slot]); }
      if (ew == 0) {
        if (!ptx::mbar_wait_relaxed(&red_bar[slot], red_phase, abort_flag, P.wait_limit)) { ok = false; break; }
        if (lane == 0 && dp_in_range(it.pidx + int(rank), (long long)P.B * P.n_per, P.dev_status)) {
          float s = 0.f;
#pragma unroll
          for (int e = 0; e < kEpiWarps; ++e) s += epi_red[slot * kEpiWarps + e];
          P.partials[it.pidx + int(rank)] = (it.ti == it.tj) ? s : 2.f * s;
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
  ptx::cluster_sync_all();        // neither CTA leaves while the partner may still use its memory
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace

dp_status launch_ghost_norm_pair(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                                 float* partials, int* dev_status, cudaStream_t st) {
  if (first_use_on_this_device(reinterpret_cast<const void*>(&ghost_norm_pair_kernel)))
    DP_CUDA_OK(cudaFuncSetAttribute(ghost_norm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kSmemBytes));
  const int nt = ceil_div(T, kTile2);
  for (size_t g0 = 0; g0 < plan.ghost_layers.size(); g0 += kGhostMaxLayers) {
    const size_t g1 = std::min(plan.ghost_layers.size(), g0 + kGhostMaxLayers);
    PairParams P;
    memset(&P, 0, sizeof(P));
    int items = 0;
    for (size_t g = g0; g < g1; ++g) {
      const int li = plan.ghost_layers[g];
      const dp_linear_desc& L = layers[li];
      dp_status s = make_tmap_bf16_3d(&P.tmA[g - g0], L.A, L.lda, L.d, T, B, kKStep, kRows);
      if (s != DP_OK) return s;
      s = make_tmap_bf16_3d(&P.tmG[g - g0], L.G, L.ldg, L.p, T, B, kKStep, kRows);
      if (s != DP_OK) return s;
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
    const int units = std::min(items, sm_count() / 2);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * units, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    DP_CUDA_OK(cudaLaunchKernelEx(&cfg, ghost_norm_pair_kernel, P));
    ++g_kernel_launches;
  }
  return DP_OK;
}

}  // namespace dpg
