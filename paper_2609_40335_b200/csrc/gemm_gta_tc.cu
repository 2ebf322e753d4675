// G^T A on tcgen05 tensor cores: the contraction over tokens shared by
//   (a) the clipped gradient sum  out = beta*out + sum_i R_i G_i^T A_i   (inner sum of Eq. 3,
//       R_i of Eq. 7), one GEMM with M = p, N = d, K = B*T whose K rows carry R_i, and
//   (b) the DIRECT per-example norm  || G_i^T A_i ||_F^2  (Eq. 4 summed over tokens), where
//       each 128 x 256 tile of the p x d gradient lives only in tensor memory and the
//       epilogue sums its squares.
//
// Both operands are contiguous along M / N (token rows are the K dimension), so shared
// memory holds MN-major tiles: every TMA box is 64 token rows x 64 columns (128-byte rows,
// 128-byte swizzle).  A K step never straddles two examples (the tensor map is 3-D:
// column, token, example; the token tail of an example is zero-filled), so one clip factor
// applies to a whole stage: a "scaler" warp multiplies the G tile by R_i in shared memory
// (packed bf16 FMAs with R_i split into two bf16 parts) between the TMA-full and MMA-ready
// barriers; four such warps work on four consecutive stages at once.
//
// Roles per CTA (704 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 scalers,
// warps 6-21 epilogue (four per TMEM lane quarter, two 32-column chunks each; they also draw
// the fused Gaussian noise, which is latency-bound per warp -- hence so many); two TMEM
// accumulators overlap the epilogue with the next tile.
//
// Clipped sums run on CTA PAIRS (cta_group::2, cluster of 2): a 256 x 256 output tile per pair,
// each CTA loading its own 128 G rows and half of the A tile's columns, rank 0 issuing the MMAs
// for both, stage-free and accumulator-ready signals multicast to both CTAs by tcgen05.commit,
// scaler and epilogue warps of rank 1 arriving on rank 0's barriers.  The DIRECT-norm variant
// stays on single CTAs.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstring>

#include "dp_common.cuh"
#include "gemm_gta.cuh"
#include "noise_device.cuh"
#include "ptx_sm100.cuh"
#include "tma_host.cuh"

namespace dpg {

namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kBoxBytes = kBK * 128;                // kBK token rows x 128 bytes
constexpr int kGBytes = (kBM / 64) * kBoxBytes;     // 16 KiB: this CTA's 128 rows of the G tile

// Tile geometry.  Single CTA: 128 x 256 output tile, the CTA loads all 256 columns of the A
// tile (48 KiB per stage, 4 stages).  CTA pair (cta_group::2): 256 x 256 output tile per pair;
// each CTA loads its own 128 G rows and HALF of the A tile's columns (32 KiB per stage, 7
// stages: all the shared memory there is -- the ring is latency-bound, 7 stages measured 973
// TFLOP/s where 6 gave 895; 32- and 128-row K steps were both slower), the pair's MMA reads
// both halves -- a third less operand traffic per flop.
template <bool kPair>
struct Geo {
  static constexpr int kAColsPerCta = kPair ? kBN / 2 : kBN;
  static constexpr int kABytes = (kAColsPerCta / 64) * kBoxBytes;
  static constexpr int kStageBytes = kGBytes + kABytes;
  static constexpr int kStages = kPair ? 7 : 4;
  static constexpr int kTileM = kPair ? 2 * kBM : kBM;       // output rows per work item
  static constexpr size_t kSmemBytes = size_t(kStages) * kStageBytes + 1024 + 1024;
};
constexpr int kProducerAWarp = 2;                    // warp 0 loads G, warp 2 loads A, warp 1 issues MMAs
constexpr int kScalerWarp0 = 3;
constexpr int kScalerWarps = 4;
constexpr int kEpiWarp0 = kScalerWarp0 + kScalerWarps;   // first epilogue warp
constexpr int kEpiWarps = 16;         // kEpiWarps/4 per TMEM lane quarter (column groups)
constexpr int kThreads = (kEpiWarp0 + kEpiWarps) * 32;
constexpr int kTmemCols = 512;                      // 2 accumulators x 256 columns

struct __align__(64) GtaParams {
  CUtensorMap tmG[kGtaMaxLayers];
  CUtensorMap tmA[kGtaMaxLayers];
  GtaLayer layer[kGtaMaxLayers];
  int n_layers;
  int B, T, tsteps;          // tsteps = ceil(T / 64) K steps per example
  int total_items;
  const float* clip;         // [B] R_i (scale mode)
  uint32_t noise_k0, noise_k1, noise_step;   // Gaussian stream of the fused noise (per-layer id)
  const uint32_t* step_dev;  // optional device counter added to noise_step
  float noise_scale;
  float* sq_partials;        // [B][n_per] (square-sum mode)
  int n_per;
  int* dev_status;
  long long wait_limit;      // cycles a barrier wait may take before the CTA gives up
};
static_assert(sizeof(GtaParams) <= 32000, "kernel parameter block too large");

struct Item {
  int layer, tm, tn, k0, k1, split, example;
};

template <bool kSqsum>
__device__ __forceinline__ Item decode_item(const GtaParams& P, int item) {
  Item it;
  int l = 0;
  while (l + 1 < P.n_layers && item >= P.layer[l + 1].item_begin) ++l;
  const GtaLayer& L = P.layer[l];
  int local = item - L.item_begin;
  it.layer = l;
  it.tn = local % L.tiles_n; local /= L.tiles_n;
  it.tm = local % L.tiles_m; local /= L.tiles_m;
  if (kSqsum) {
    it.example = local; it.split = 0;
    it.k0 = local * P.tsteps; it.k1 = it.k0 + P.tsteps;
  } else {
    it.example = -1; it.split = local;
    it.k0 = local * L.ksteps_per_split;
    it.k1 = min(it.k0 + L.ksteps_per_split, P.B * P.tsteps);
  }
  return it;
}

// Partial in-register transpose of a 32 x 32 tile held one row per lane (v[c] = column c): the
// upper three lane bits are exchanged with the upper three register bits (three butterfly stages
// of 16 exchanges).  Afterwards lane l holds, in v[4i .. 4i+3], columns 4(l>>2) .. +3 of row
// 4i + (l&3): four consecutive columns per register quad, and the 32 lanes of quad i cover rows
// 4i .. 4i+3 completely -- one float4 store per quad writes four whole 128-byte lines.
__device__ __forceinline__ void warp_transpose_quads(float (&v)[32], int lane) {
#pragma unroll
  for (int d = 16; d >= 4; d >>= 1) {
    const bool up = (lane & d) != 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      if ((j & d) == 0) {
        const float send = up ? v[j] : v[j + d];
        const float recv = __shfl_xor_sync(0xffffffffu, send, d);
        if (up) v[j] = recv; else v[j + d] = recv;
      }
    }
  }
}

template <bool kScale, bool kSqsum, bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
gemm_gta_kernel(const __grid_constant__ GtaParams P) {
  static_assert(kScale || !kPair, "CTA pairs need the scaler warps' cross-CTA stage hand-off");
  constexpr int kStages = Geo<kPair>::kStages;
  constexpr int kStageBytes = Geo<kPair>::kStageBytes;
  constexpr int kTileM = Geo<kPair>::kTileM;
  constexpr int kPeers = kPair ? 2 : 1;
  // pair: rank 0 issues the MMAs; both CTAs walk the same list of work items
  const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;
  const int first_item = kPair ? int(blockIdx.x >> 1) : int(blockIdx.x);
  const int item_stride = kPair ? int(gridDim.x >> 1) : int(gridDim.x);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + size_t(kStages) * kStageBytes);
  uint64_t* full = bars;                      // both producers' TMA loads landed
  uint64_t* ready = bars + kStages;           // G tile scaled in both CTAs (scale mode; rank 0's copy)
  uint64_t* empty = bars + 2 * kStages;       // MMAs retired
  uint64_t* acc_full = bars + 3 * kStages;    // [2]
  uint64_t* acc_empty = acc_full + 2;         // [2]
  uint64_t* mma_done = acc_empty + 2;         // only used when the MMA issuer gives up
  uint64_t* red_bar = mma_done + 1;           // [4] epilogue warps -> epilogue warp 0 (square-sum mode)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(red_bar + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* epi_red = reinterpret_cast<float*>(tmem_slot + 2);   // [4][kEpiWarps]
  uint32_t* sink = reinterpret_cast<uint32_t*>(epi_red + 4 * kEpiWarps);   // [kStages] written by st.async, never read

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t tiles_a = ptx::smem_u32(tiles);
  const uint32_t full_a = ptx::smem_u32(full), ready_a = ptx::smem_u32(ready), empty_a = ptx::smem_u32(empty);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(&full[s], 2);             // the G producer and the A producer
      // pair: rank 0's scaler warp arrives (and announces 4 bytes), rank 1's sends those 4 bytes
      ptx::mbar_init(&ready[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&acc_full[b], 1);
      ptx::mbar_init(&acc_empty[b], kEpiWarps * kPeers);    // epilogue warps of both CTAs
    }
    ptx::mbar_init(mma_done, 1);
    for (int b = 0; b < 4; ++b) ptx::mbar_init(&red_bar[b], kEpiWarps);
    *abort_flag = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 1) {
    if (kPair) { ptx::tmem_alloc_pair(tmem_slot, kTmemCols); ptx::tmem_relinquish_pair(); }
    else { ptx::tmem_alloc(tmem_slot, kTmemCols); ptx::tmem_relinquish(); }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (kPair) ptx::cluster_sync_all();     // the partner's barriers exist before anyone arrives on them
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == kProducerAWarp) {
    // ------------------------------------------------------------- TMA producers
    // Two threads in two warps: one loads this CTA's G rows, the other its A columns.  The time
    // a producer needs per stage is part of every stage's round trip, so the work is halved and
    // the loop is kept to a few instructions (32-bit shared addresses, running example / token
    // counters instead of a division).
    if (lane == 0) {
      const bool is_a = (warp != 0);
      constexpr int kBoxes = kBM / 64;
      constexpr int kBoxesA = Geo<kPair>::kAColsPerCta / 64;
      const uint32_t my_bytes = is_a ? uint32_t(Geo<kPair>::kABytes) : uint32_t(kGBytes);
      const int nbox = is_a ? kBoxesA : kBoxes;
      uint32_t stage = 0, phase = 0, issued = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride) {
        const Item it = decode_item<kSqsum>(P, item);
        const uint64_t tm = reinterpret_cast<uint64_t>(is_a ? &P.tmA[it.layer] : &P.tmG[it.layer]);
        // first column of this CTA's part of the tile: its G rows, or its share of the A columns
        const int c0 = is_a ? it.tn * kBN + int(rank) * Geo<kPair>::kAColsPerCta
                            : it.tm * kTileM + int(rank) * kBM;
        int ex = it.k0 / P.tsteps, ts = it.k0 - ex * P.tsteps;
        for (int ks = it.k0; ks < it.k1; ++ks) {
          if (!ptx::mbar_wait_a(empty_a + 8 * stage, phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
          const uint32_t bar = full_a + 8 * stage;
          const uint32_t dst = tiles_a + stage * kStageBytes + (is_a ? kGBytes : 0);
          ptx::mbar_arrive_expect_tx_a(bar, my_bytes);
          for (int j = 0; j < nbox; ++j)
            ptx::tma_load_3d_a(dst + j * kBoxBytes, tm, bar, c0 + j * 64, ts * kBK, ex);
          ++issued;
          if (++ts == P.tsteps) { ts = 0; ++ex; }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
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
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16_f32(kTileM, kBN, 1, 1);
      // MN-major, 128-byte swizzle: 64-column chunks are one box (8 KiB) apart, groups of
      // 8 token rows are 1 KiB apart.  Only the 14-bit start address in the low word changes.
      constexpr uint64_t dbase = ptx::smem_desc_base(kBoxBytes, 1024, ptx::SWIZZLE_128B);
      constexpr uint32_t desc_hi = uint32_t(dbase >> 32);
      const uint32_t desc_lo0 = uint32_t(dbase) | ((tiles_a >> 4) & 0x3FFF);
      const uint32_t go_a = kScale ? ready_a : full_a;
      uint32_t stage = 0, phase = 0, n_item = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride, ++n_item) {
        const Item it = decode_item<kSqsum>(P, item);
        const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
        if (!(kPair ? ptx::mbar_wait_cluster(&acc_empty[buf], acc_phase ^ 1, abort_flag, P.wait_limit)
                    : ptx::mbar_wait(&acc_empty[buf], acc_phase ^ 1, abort_flag, P.wait_limit))) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * kBN;
        uint32_t accum = 0;
        for (int ks = it.k0; ks < it.k1; ++ks) {
          if (!(kPair ? ptx::mbar_wait_cluster_a(go_a + 8 * stage, phase, abort_flag, P.wait_limit)
                      : ptx::mbar_wait_a(go_a + 8 * stage, phase, abort_flag, P.wait_limit))) { ok = false; break; }
          ptx::tc_fence_after();
          const uint32_t lo_g = desc_lo0 + stage * (kStageBytes >> 4);
          const uint32_t lo_a = lo_g + (kGBytes >> 4);
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk) {
            // 16 token rows further = two 1 KiB row groups
            if (kPair) ptx::mma_bf16_ss_pair_lh(d_tmem, lo_g + kk * 128, lo_a + kk * 128, desc_hi, idesc, accum);
            else ptx::mma_bf16_ss_lh(d_tmem, lo_g + kk * 128, lo_a + kk * 128, desc_hi, idesc, accum);
            accum = 1;
          }
          // stage reusable in both CTAs once these MMAs retire
          if (kPair) ptx::mma_commit_pair_a(empty_a + 8 * stage, 3);
          else ptx::mma_commit_a(empty_a + 8 * stage);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) {
          if (kPair) ptx::mma_commit_pair(&acc_full[buf], 3);
          else ptx::mma_commit(&acc_full[buf]);
        }
      }
      if (!ok) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
        ptx::drain_issued_mmas(mma_done, kPair);
      }
    }
  } else if (warp < kEpiWarp0) {
    // ------------------------------------------------------------------ scalers
    if (kScale) {
      // Each scaler warp owns every kScalerWarps-th K step, so kScalerWarps stages are scaled
      // concurrently: the per-stage latency (shared-memory round trip, proxy fence, barrier
      // hand-off) is overlapped instead of serialised.
      //
      // Hand-off to the MMA issuer (rank 0).  Rank 0's warp arrives on its own `ready` barrier
      // and announces 4 more bytes; rank 1's warp delivers those 4 bytes with an asynchronous
      // store into rank 0's shared memory whose completion on the barrier is a release at
      // cluster scope: the scaled tile it wrote (made visible to the tensor core's proxy by the
      // fence before) is ordered before the MMAs that rank 0 issues after its acquire.
      const int sw = warp - kScalerWarp0;
      const uint32_t ready_remote = kPair ? ptx::mapa_u32(ready_a, 0) : 0u;
      const uint32_t sink_remote = kPair ? ptx::mapa_u32(ptx::smem_u32(sink), 0) : 0u;
      uint32_t cnt = 0;
      bool ok = true;
      for (int item = first_item; item < P.total_items && ok; item += item_stride) {
        const Item it = decode_item<kSqsum>(P, item);
        const bool scale_here = P.clip && !P.layer[it.layer].prescaled;
        // first K step of this item that belongs to this warp
        int ks = it.k0 + int((uint32_t(sw) + kScalerWarps - cnt % kScalerWarps) % kScalerWarps);
        uint32_t c = cnt + uint32_t(ks - it.k0);
        // no scaling here when the operand arrives scaled: clip == NULL (the split fp32 path) or a
        // layer whose narrow operand was multiplied by R_i in a pass of its own (see prescale)
        float r_next = (scale_here && ks < it.k1) ? __ldg(P.clip + ks / P.tsteps) : 1.f;
        for (; ks < it.k1; ks += kScalerWarps, c += kScalerWarps) {
          const float r = r_next;
          // the factor of this warp's next K step is fetched before the waits, off the stage's path
          if (scale_here && ks + kScalerWarps < it.k1) r_next = __ldg(P.clip + (ks + kScalerWarps) / P.tsteps);
          const uint32_t stage = c % kStages, fill = c / kStages, phase = fill & 1u;
          // A warp hops between stages, so it has not seen the previous fill of this one, and the
          // parity of `full` alone cannot tell "fill n landed" from "fill n-1 still in flight".
          // Waiting first until the MMAs have retired fill n-1 (the same condition the producers
          // wait for before they issue fill n, so no time is lost) leaves only "fill n pending"
          // or "fill n landed".
          if (fill > 0 && !ptx::mbar_wait_a(empty_a + 8 * stage, phase ^ 1, abort_flag, P.wait_limit)) { ok = false; break; }
          if (!ptx::mbar_wait_a(full_a + 8 * stage, phase, abort_flag, P.wait_limit)) { ok = false; break; }
          if (r != 1.0f) {
            // r = r_hi + r_lo with both parts in bf16 (16 mantissa bits in total); g*r is formed
            // as fma(g, r_hi, g*r_lo) on packed bf16 pairs: one rounding of the exact g*r_hi plus
            // a tiny correction, i.e. the correctly rounded bf16 product up to 2^-17 relative.
            const __nv_bfloat16 rh = __float2bfloat16_rn(r);
            const __nv_bfloat16 rl = __float2bfloat16_rn(r - __bfloat162float(rh));
            const __nv_bfloat162 rh2 = __halves2bfloat162(rh, rh), rl2 = __halves2bfloat162(rl, rl);
            // kChunks 16-byte chunks per lane, eight at a time
            constexpr int kChunks = kGBytes / 16 / 32;
            uint4* g = reinterpret_cast<uint4*>(tiles + size_t(stage) * kStageBytes) + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < kChunks; c0 += 8) {
              uint4 v[8];
#pragma unroll
              for (int q = 0; q < 8; ++q) v[q] = g[(c0 + q) * 32];
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                __nv_bfloat162* w = reinterpret_cast<__nv_bfloat162*>(&v[q]);
#pragma unroll
                for (int e = 0; e < 4; ++e) w[e] = __hfma2(w[e], rh2, __hmul2(w[e], rl2));
                g[(c0 + q) * 32] = v[q];
              }
            }
            ptx::fence_proxy_async_smem();
          }
          __syncwarp();
          if (lane == 0) {
            if (!kPair) ptx::mbar_arrive(&ready[stage]);
            else if (rank == 0) ptx::mbar_arrive_expect_tx_a(ready_a + 8 * stage, 4);
            else ptx::st_async_signal_a(ready_remote + 8 * stage, sink_remote + 4 * stage);
          }
        }
        cnt += uint32_t(it.k1 - it.k0);
      }
      if (!ok && lane == 0) {
        *abort_flag = 1;
        if (P.dev_status) atomicOr(P.dev_status, DP_DEV_TIMEOUT);
      }
    }
  } else {
    // ----------------------------------------------------------------- epilogue
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int ew = warp - kEpiWarp0;
    // this warp's 32-column chunks: the 8 chunks are dealt to the kEpiWarps/4 column groups
    constexpr int kGroups = kEpiWarps / 4;
    const int c_lo = ((ew >> 2) * (kBN / 32)) / kGroups, c_hi = (((ew >> 2) + 1) * (kBN / 32)) / kGroups;
    uint32_t n_item = 0;
    bool ok = true;
    for (int item = first_item; item < P.total_items && ok; item += item_stride, ++n_item) {
      const Item it = decode_item<kSqsum>(P, item);
      const GtaLayer& L = P.layer[it.layer];
      const uint32_t buf = n_item & 1, acc_phase = (n_item >> 1) & 1;
      if (!ptx::mbar_wait_relaxed(&acc_full[buf], acc_phase, abort_flag, P.wait_limit)) { ok = false; break; }
      ptx::tc_fence_after();
      const uint32_t t0 = tmem_base + (uint32_t(q * 32) << 16) + buf * kBN;
      const int row = it.tm * kTileM + int(rank) * kBM + q * 32 + lane;
      if (kSqsum) {
        float acc = 0.f;
#pragma unroll 1
        for (int c = c_lo; c < c_hi; ++c) {
          uint32_t r[32];
          ptx::tmem_ld_32x32b_x32(t0 + c * 32, r);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) { const float v = __uint_as_float(r[j]); acc = fmaf(v, v, acc); }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kPair) ptx::mbar_arrive_cluster(&acc_empty[buf], 0);
          else ptx::mbar_arrive(&acc_empty[buf]);
        }
        // the warps' sums meet through an mbarrier with a bounded wait (no blocking named
        // barrier: a warp that gave up never arrives); four slots, since the other warps can run
        // at most two items ahead of a waiting warp 0 (they need its acc_empty arrivals)
        acc = warp_sum(acc);
        const uint32_t slot = n_item & 3, red_phase = (n_item >> 2) & 1;
        if (lane == 0) { epi_red[slot * kEpiWarps + ew] = acc; ptx::mbar_arrive(&red_bar[slot]); }
        if (ew == 0) {
          if (!ptx::mbar_wait_relaxed(&red_bar[slot], red_phase, abort_flag, P.wait_limit)) { ok = false; break; }
          const long long slot_idx = (long long)it.example * P.n_per + L.col_begin + it.tm * L.tiles_n + it.tn;
          if (lane == 0 && dp_in_range(slot_idx, (long long)P.B * P.n_per, P.dev_status)) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < kEpiWarps; ++e) s += epi_red[slot * kEpiWarps + e];
            P.sq_partials[size_t(it.example) * P.n_per + L.col_begin + it.tm * L.tiles_n + it.tn] = s;
          }
        }
      } else {
        // destination: the layer's output (no K split) or this split's partial plane
        float* dst;
        long long ld;
        float beta;
        if (L.nsplit == 1) { dst = L.out; ld = L.ldo; beta = L.beta; }
        else { dst = L.partial + size_t(it.split) * size_t(L.M) * L.N; ld = L.N; beta = 0.f; }
        const bool vec_ok = ((ld & 3) == 0) && ((reinterpret_cast<uintptr_t>(dst) & 15) == 0);
        // fused Gaussian mechanism (Eq. 3): only on the final destination, never on a K-split plane
        const bool noisy = (L.noise_amp >= 0.f) && (L.nsplit == 1);
        const NoiseKey nkey{P.noise_k0, P.noise_k1, L.tensor_id, effective_step(P.noise_step, P.step_dev)};
#pragma unroll 1
        for (int c = c_lo; c < c_hi; ++c) {
          uint32_t r[32];
          ptx::tmem_ld_32x32b_x32(t0 + c * 32, r);
          ptx::tmem_ld_wait();
          const int col0 = it.tn * kBN + c * 32;
          const int row_base = row - lane;                   // first row of this warp's 32
          if (row_base < L.M && col0 < L.N) {                // the same for the whole warp
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
            if (row < L.M) {
              const bool full32 = col0 + 32 <= L.N;
              if (beta != 0.f) {
                const float* o = dst + size_t(row) * ld + col0;
                if (vec_ok && full32) {
#pragma unroll
                  for (int j = 0; j < 8; ++j) {
                    const float4 old = *reinterpret_cast<const float4*>(o + 4 * j);
                    v[4 * j] += old.x; v[4 * j + 1] += old.y; v[4 * j + 2] += old.z; v[4 * j + 3] += old.w;
                  }
                } else {
#pragma unroll
                  for (int j = 0; j < 32; ++j) if (col0 + j < L.N) v[j] += o[j];
                }
              }
              if (noisy) {
                const unsigned long long j0 = (unsigned long long)row * L.N + col0;   // stream index
                // N is a multiple of 4 here (the host fuses only such layers), so the Philox
                // counters of this thread's 32 columns never straddle a row
#pragma unroll
                for (int qd = 0; qd < 8; ++qd) {
                  if (col0 + 4 * qd < L.N) {
                    float z[4];
                    normals4((j0 >> 2) + qd, nkey, z);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                      v[4 * qd + e] = noised(v[4 * qd + e], z[e], L.noise_amp, P.noise_scale);
                  }
                }
              }
            }
            // Stores by whole lines: with one row per lane a warp store would touch 32 different
            // 128-byte lines, 16 bytes each -- measured, those write requests took a fifth of the
            // kernel's throughput away from the operand loads.  After the partial transpose every
            // float4 store of the warp writes four complete rows of this 32-column chunk.
            warp_transpose_quads(v, lane);
            const int colq = col0 + 4 * (lane >> 2);         // this lane's four columns
            const int rsub = lane & 3;
            if (vec_ok && col0 + 32 <= L.N) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int rr = row_base + 4 * i + rsub;
                if (rr < L.M)
                  __stcs(reinterpret_cast<float4*>(dst + size_t(rr) * ld + colq),
                         make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
              }
            } else {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int rr = row_base + 4 * i + rsub;
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (rr < L.M && colq + e < L.N) dst[size_t(rr) * ld + colq + e] = v[4 * i + e];
              }
            }
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kPair) ptx::mbar_arrive_cluster(&acc_empty[buf], 0);
          else ptx::mbar_arrive(&acc_empty[buf]);
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
  // pair: neither CTA may leave while the partner can still read its shared memory or arrive on
  // its barriers (every wait above is bounded, so both always get here)
  if (kPair) ptx::cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after();
    if (kPair) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// out = beta*out + sum over K splits of the partial planes, in split order
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, int nsplit, int M, int N,
                                     float* __restrict__ out, long long ldo, float beta) {
  const size_t total = size_t(M) * N;
  for (size_t e = size_t(blockIdx.x) * blockDim.x + threadIdx.x; e < total;
       e += size_t(gridDim.x) * blockDim.x) {
    const int r = int(e / N), c = int(e - size_t(r) * N);
    float s = 0.f;
    for (int k = 0; k < nsplit; ++k) s += partial[size_t(k) * total + e];
    float* o = out + size_t(r) * ldo + c;
    *o = (beta != 0.f) ? (*o + s) : s;
  }
}

// out[r, :] = bf16(R_{r / T} * src[r, :]) for the B*T token rows of a narrow operand
__global__ void __launch_bounds__(256)
prescale_rows_kernel(const __nv_bfloat16* __restrict__ src, long long lds, __nv_bfloat16* __restrict__ dst,
                     int cp, long long rows, int T, int c, const float* __restrict__ clip) {
  const int per_row = cp >> 3;                      // 16-byte chunks per output row
  const long long total = rows * per_row;
  const bool vec = ((reinterpret_cast<uintptr_t>(src) & 15) == 0) && ((lds & 7) == 0);
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const long long r = e / per_row;
    const int c0 = int(e - r * per_row) << 3;
    float v[8];
    load8<__nv_bfloat16>(src + r * lds + c0, c - c0, vec, v);   // columns >= c read as zero
    const float f = clip[r / T];
    uint4 o;
    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int k = 0; k < 4; ++k) o2[k] = __floats2bfloat162_rn(v[2 * k] * f, v[2 * k + 1] * f);
    *reinterpret_cast<uint4*>(dst + r * cp + c0) = o;
  }
}

// A layer whose narrow operand is at most a twentieth of its input bytes (the LM head: d = 768
// against p = 50257) gets that operand multiplied by R_i in a pass of its own -- a few
// microseconds -- and then runs through the GEMM unscaled: the in-pipeline scaling costs
// shared-memory bandwidth on EVERY K step of every tile of the wide operand, the copy does not.
inline bool prescale_layer(const dp_linear_desc& L) {
  return 20LL * std::min(L.d, L.p) <= (long long)L.d + L.p;
}
inline size_t prescale_bytes(const dp_linear_desc& L, int B, int T) {
  const int cp = (std::min(L.d, L.p) + 7) / 8 * 8;
  return align_up(size_t(B) * T * cp * 2, 256);
}

// The clipped sum always runs with kScale = true: on CTA pairs the scaler warps are also what
// tells rank 0's MMA issuer that BOTH CTAs' halves of a stage have landed.  (kScale = false is
// for the single-CTA DIRECT-norm kernel only; a pair kernel without the scalers' hand-off would
// let the issuer run ahead of the partner's loads and re-arm a stage barrier in mid-phase.)
constexpr bool kClipScale = true;

constexpr bool kUsePair = true;

template <bool kScale, bool kSqsum, bool kPair>
dp_status set_attr_once() {
  if (first_use_on_this_device(reinterpret_cast<const void*>(&gemm_gta_kernel<kScale, kSqsum, kPair>)))
    DP_CUDA_OK(cudaFuncSetAttribute(gemm_gta_kernel<kScale, kSqsum, kPair>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)Geo<kPair>::kSmemBytes));
  return DP_OK;
}

// Launch on `units` persistent CTAs (single) or CTA pairs (cluster of 2).
template <bool kScale, bool kSqsum, bool kPair>
dp_status launch_gta(const GtaParams& P, int units, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kPair ? 2 * units : units, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = Geo<kPair>::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kPair ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  DP_CUDA_OK(cudaLaunchKernelEx(&cfg, gemm_gta_kernel<kScale, kSqsum, kPair>, P));
  ++g_kernel_launches;
  return DP_OK;
}

}  // namespace

// K-split factor shared by all layers of one grouped call: 1 when the output tiles alone give
// every SM at least two items, otherwise enough splits to get there (>= 4 K steps per split).
int gta_choose_nsplit(const dp_linear_desc* layers, int n_layers, int B, int T, int sms) {
  long long tiles = 0;
  for (int l = 0; l < n_layers; ++l)
    tiles += (long long)ceil_div(layers[l].p, Geo<kUsePair>::kTileM) * ceil_div(layers[l].d, kBN);
  const int ksteps = B * ceil_div(T, kBK);
  const int units = kUsePair ? sms / 2 : sms;          // persistent CTAs or CTA pairs
  if (tiles >= 2LL * units) return 1;
  long long ns = std::max<long long>(1, (2LL * units) / std::max<long long>(tiles, 1));
  ns = std::min<long long>(ns, std::max(1, ksteps / 4));
  return (int)std::max<long long>(1, ns);
}

size_t gta_partial_bytes(const dp_linear_desc* layers, int n_layers, int B, int T, int sms) {
  const int ns = gta_choose_nsplit(layers, n_layers, B, T, sms);
  size_t n = 0;
  for (int l = 0; l < n_layers; ++l) {
    if (ns > 1) n += align_up(size_t(ns) * size_t(layers[l].p) * size_t(layers[l].d) * sizeof(float), 256);
    if (prescale_layer(layers[l])) n += prescale_bytes(layers[l], B, T);
  }
  return n;
}

dp_status launch_clip_accumulate_tc(const dp_linear_desc* layers, int n_layers, int B, int T,
                                    const float* clip, float* const* outs, const int64_t* ldos,
                                    float beta, const GtaNoise* noise, float* partial_ws,
                                    int* dev_status, cudaStream_t st) {
  dp_status s = set_attr_once<kClipScale, false, kUsePair>();
  if (s != DP_OK) return s;
  const int sms = sm_count();
  const int tsteps = ceil_div(T, kBK);
  const int ksteps = B * tsteps;
  int nsplit = gta_choose_nsplit(layers, n_layers, B, T, sms);
  const int kps = ceil_div(ksteps, nsplit);
  nsplit = ceil_div(ksteps, kps);                       // drop empty trailing splits
  char* pw = reinterpret_cast<char*>(partial_ws);
  char* pre = pw;                                       // pre-scaled copies sit behind the K-split planes
  if (pw && nsplit > 1)
    for (int l = 0; l < n_layers; ++l)
      pre += align_up(size_t(nsplit) * size_t(layers[l].p) * size_t(layers[l].d) * sizeof(float), 256);
  for (int g0 = 0; g0 < n_layers; g0 += kGtaMaxLayers) {
    const int g1 = std::min(n_layers, g0 + kGtaMaxLayers);
    GtaParams P;
    memset(&P, 0, sizeof(P));
    int items = 0;
    for (int g = g0; g < g1; ++g) {
      dp_linear_desc D = layers[g];
      GtaLayer& L = P.layer[g - g0];
      L.prescaled = 0;
      if (clip && pw && prescale_layer(D)) {
        // R_i onto the narrow operand, into the workspace; the GEMM then reads the copy
        const bool narrow_a = D.d <= D.p;
        const int c = narrow_a ? D.d : D.p, cp = (c + 7) / 8 * 8;
        __nv_bfloat16* copy = reinterpret_cast<__nv_bfloat16*>(pre);
        pre += prescale_bytes(D, B, T);
        const long long rows = (long long)B * T;
        const int blocks = (int)std::min<long long>((rows * (cp >> 3) + 255) / 256, (long long)sms * 16);
        prescale_rows_kernel<<<blocks, 256, 0, st>>>(
            static_cast<const __nv_bfloat16*>(narrow_a ? D.A : D.G), narrow_a ? D.lda : D.ldg, copy, cp,
            rows, T, c, clip);
        DP_LAUNCH_OK();
        if (narrow_a) { D.A = copy; D.lda = cp; } else { D.G = copy; D.ldg = cp; }
        L.prescaled = 1;
      }
      s = make_tmap_bf16_3d(&P.tmG[g - g0], D.G, D.ldg, D.p, T, B, 64, kBK);
      if (s != DP_OK) return s;
      s = make_tmap_bf16_3d(&P.tmA[g - g0], D.A, D.lda, D.d, T, B, 64, kBK);
      if (s != DP_OK) return s;
      L.out = outs[g]; L.ldo = ldos[g]; L.beta = beta;
      L.M = D.p; L.N = D.d;
      L.tiles_m = ceil_div(D.p, Geo<kUsePair>::kTileM); L.tiles_n = ceil_div(D.d, kBN);
      L.nsplit = nsplit; L.ksteps_per_split = kps;
      L.partial = nullptr;
      if (nsplit > 1) {
        L.partial = reinterpret_cast<float*>(pw);
        pw += align_up(size_t(nsplit) * size_t(D.p) * size_t(D.d) * sizeof(float), 256);
      }
      L.item_begin = items; L.col_begin = 0;
      // noise is drawn in the epilogue when the layer is not K-split and its width is a
      // multiple of 4; otherwise a stand-alone pass follows (negative amp: no fused noise)
      const bool fuse = noise && nsplit == 1 && (D.d % 4 == 0);
      L.noise_amp = fuse ? noise->amp : -1.f;
      L.tensor_id = noise ? noise->tensor_ids[g] : 0u;
      items += L.tiles_m * L.tiles_n * nsplit;
    }
    if (noise) {
      P.noise_k0 = uint32_t(noise->seed); P.noise_k1 = uint32_t(noise->seed >> 32);
      P.noise_step = noise->step; P.noise_scale = noise->scale;
      P.step_dev = g_step_dev;
    }
    P.n_layers = g1 - g0; P.B = B; P.T = T; P.tsteps = tsteps;
    P.total_items = items;
    P.clip = clip;
    P.dev_status = dev_status;
    P.wait_limit = g_wait_limit;
    const int units = std::min(items, kUsePair ? sms / 2 : sms);
    s = launch_gta<kClipScale, false, kUsePair>(P, units, st);
    if (s != DP_OK) return s;
    for (int g = g0; g < g1; ++g) {
      const GtaLayer& L = P.layer[g - g0];
      if (nsplit > 1) {
        const size_t total = size_t(L.M) * L.N;
        const int blocks = (int)std::min<size_t>((total + 255) / 256, size_t(sms) * 8);
        splitk_reduce_kernel<<<blocks, 256, 0, st>>>(L.partial, nsplit, L.M, L.N, L.out, L.ldo, beta);
        DP_LAUNCH_OK();
      }
      if (noise && L.noise_amp < 0.f) {        // not fused for this layer: stand-alone pass
        const dp_status ns = launch_add_noise(L.out, L.M, L.N, L.ldo, false, noise->amp,
                                              noise->scale, noise->seed, noise->tensor_ids[g],
                                              noise->step, st);
        if (ns != DP_OK) return ns;
      }
    }
  }
  return DP_OK;
}


dp_status launch_direct_norm_tc(const dp_linear_desc* layers, const GhostPlan& plan, int B, int T,
                                float* partials, int* dev_status, cudaStream_t st) {
  dp_status s = set_attr_once<false, true, false>();
  if (s != DP_OK) return s;
  const int sms = sm_count();
  for (size_t g0 = 0; g0 < plan.direct_layers.size(); g0 += kGtaMaxLayers) {
    const size_t g1 = std::min(plan.direct_layers.size(), g0 + kGtaMaxLayers);
    GtaParams P;
    memset(&P, 0, sizeof(P));
    int items = 0;
    for (size_t g = g0; g < g1; ++g) {
      const int li = plan.direct_layers[g];
      const dp_linear_desc& D = layers[li];
      s = make_tmap_bf16_3d(&P.tmG[g - g0], D.G, D.ldg, D.p, T, B, 64, kBK);
      if (s != DP_OK) return s;
      s = make_tmap_bf16_3d(&P.tmA[g - g0], D.A, D.lda, D.d, T, B, 64, kBK);
      if (s != DP_OK) return s;
      GtaLayer& L = P.layer[g - g0];
      L.M = D.p; L.N = D.d;
      L.tiles_m = plan.direct[li].tiles_m; L.tiles_n = plan.direct[li].tiles_n;
      L.nsplit = 1; L.ksteps_per_split = 0;
      L.col_begin = plan.direct[li].col_begin;
      L.item_begin = items;
      items += B * L.tiles_m * L.tiles_n;
    }
    P.n_layers = int(g1 - g0);
    P.B = B; P.T = T; P.tsteps = ceil_div(T, kBK);
    P.total_items = items;
    P.sq_partials = partials; P.n_per = plan.n_per;
    P.dev_status = dev_status;
    P.wait_limit = g_wait_limit;
    s = launch_gta<false, true, false>(P, std::min(items, sms), st);
    if (s != DP_OK) return s;
  }
  return DP_OK;
}

}  // namespace dpg
