// Kernel 2 (paired form): block-scaled MXFP4 x MXFP4 GEMM with two CTAs per 256 x 256 output tile
// (paper Sec. 1 / Sec. 4.2: W4A4, y = Q(xR) Q(WR)^T; fp32 accumulation, bf16 or fp32 output).
//
// Why pairs: one CTA computing a 128 x 256 tile pulls (128 + 256) x 128 bytes of codes from L2
// per 256-deep K step, 341 flop per byte, and the tensor pipe waits for L2 half of the time.  With
// tcgen05.mma.cta_group::2 the two CTAs of a cluster multiply a 256 x 256 tile together: each CTA
// loads ITS 128 rows of A and ITS 128 rows of W (plus scales) and the tensor cores read both
// halves of W across the pair, so every CTA pulls (128 + 128) x 128 bytes per step for the same
// flops — 480 flop per byte — with no multicast load anywhere.
//
// Roles in each CTA (192 threads):
//   warp 0      TMA producer for this CTA's operand halves.  All loads of both CTAs count their
//               bytes on the LEADER's "full" barrier (cp.async.bulk.tensor ... .cta_group::2).
//   warp 1      owns this CTA's TMEM.  In the leader (cluster rank 0) one thread copies the scale
//               blocks shared -> TMEM and issues the MMAs for the pair; tcgen05.commit with a
//               2-CTA mask releases the stage, or hands the accumulator over, in both CTAs.
//   warps 2..5  epilogue for this CTA's 128 rows: TMEM -> registers -> bf16 -> swizzled staging
//               -> TMA store.  "Drained" arrivals of both CTAs go to the leader's barriers.
// Accumulators: two per CTA, overlapping by 32 TMEM columns ([0,256) and [224,480)), scale columns
// at [480,504) — the same arrangement as the single-CTA kernel.
// Every mbarrier wait is bounded.  Both CTAs always reach the cluster barrier at the end, so neither
// leaves while its partner may still touch its shared memory, barriers or TMEM.
#pragma once

#include "gemm_mxfp4.cuh"

namespace bro {
namespace gemm2 {

using gemm::kChunkCols;
using gemm::kStageOutBytes;

constexpr int kBM = 128;                 // rows per CTA (256 per pair)
constexpr int kBN = 256;                 // columns per pair tile
constexpr int kBK = 256;
constexpr int kThreads = 192;
constexpr int kStages = 5;
constexpr int kATileBytes = kBM * 128;          // 16 KiB
constexpr int kBTileBytes = (kBN / 2) * 128;    // 16 KiB: this CTA's half of W
constexpr int kSfaBytes = 1024;                 // 2 blocks of 512 B (128 rows x 4 groups)
constexpr int kSfbBytes = 2048;                 // all 256 columns: 2 row blocks x 2 K blocks
constexpr int kStageBytes = kATileBytes + kBTileBytes + kSfaBytes + kSfbBytes;   // 35 KiB
constexpr int kSmemBytes = kStages * kStageBytes + 2 * kStageOutBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr int kTmemCols = 512;
constexpr int kAccStride = 224;
constexpr int kSfaCol = 480;
constexpr int kSfbCol = 488;
constexpr int kChunks = kBN / kChunkCols;
constexpr int kRasterRows = 8;           // tile rows per raster group (L2 reuse of both operands)

struct Params {
  void* y;
  int64_t M, N, ldy;
  int num_k_steps;          // ceil(K/256)
  int tiles_m, tiles_n, total_tiles;   // 256 x 256 tiles
  // Work units, as in the single-CTA kernel: units [0, full_units) are whole tiles; when the last round
  // of the grid would be less than half full, its tiles are cut into two 256 x 128 halves each.
  int full_units, total_units;
};

// ---- cluster helpers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
// Arrive on a barrier of a CTA of this cluster.  Relaxed on purpose: what the arrival reports — this
// warp's tcgen05.ld of the accumulator columns — is already complete (tcgen05.wait::ld has returned,
// the values are in registers), so nothing has to be made visible through memory; a release at cluster
// scope would first wait for every earlier memory operation of the thread, the staging-buffer stores
// and TMA stores of the tile before included, and delayed the next tile's first MMA by 0.6 us.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// 2-D tiled load into THIS CTA's shared memory whose byte count completes on an mbarrier that may
// live in the partner CTA (shared::cluster address).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair_if(uint32_t issue, uint32_t dst, const CUtensorMap* m, int x,
                                                    int y, uint32_t bar_cluster) {
  asm volatile(
      "{ .reg .pred q; setp.ne.b32 q, %5, 0;\n\t"
      "@q cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4]; }" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(bar_cluster), "r"(issue)
      : "memory");
}
// E2M1 x E2M1, K-major, UE8M0 scales, M = 256 (128 rows per CTA), N = BN.
template <int BN>
__device__ __forceinline__ constexpr uint32_t make_idesc_pair() {
  return (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) | ((uint32_t)(256 >> 4) << 24);
}

// Tile order: groups of kRasterRows tile rows, column by column inside a group, so that the pairs
// running at the same time share a few A panels and a few W panels.
// Unit index -> tile, which half of it (0 when the unit is a whole tile) and its width.
__device__ __forceinline__ void unit_tile(int u, const Params& p, int& tile, int& half, int& bn) {
  tile = u; half = 0; bn = kBN;
  if (u >= p.full_units) {
    const int idx = u - p.full_units;
    tile = p.full_units + (idx >> 1);
    half = idx & 1;
    bn = kBN / 2;
  }
}
__device__ __forceinline__ void tile_coords(int tile, const Params& p, int& tm, int& tn) {
  const int per_group = kRasterRows * p.tiles_n;
  const int g = tile / per_group;
  const int within = tile - g * per_group;
  const int rows = min(kRasterRows, p.tiles_m - g * kRasterRows);
  tn = within / rows;
  tm = g * kRasterRows + (within - tn * rows);
}

template <bool OUT_F32>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_mxfp4_pair_kernel(const __grid_constant__ CUtensorMap tma, const __grid_constant__ CUtensorMap tmw,
                       const __grid_constant__ CUtensorMap tmw_half, const __grid_constant__ CUtensorMap tmsfa,
                       const __grid_constant__ CUtensorMap tmsfb, const __grid_constant__ CUtensorMap tmy,
                       const Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = smem_base;
  const uint32_t sB = sA + kStages * kATileBytes;
  const uint32_t sSFA = sB + kStages * kBTileBytes;
  const uint32_t sSFB = sSFA + kStages * kSfaBytes;
  const uint32_t sOut = sSFB + kStages * kSfbBytes;               // 2 x 8 KiB, 1 KiB aligned
  const uint32_t bar_base = sOut + 2 * kStageOutBytes;
  const uint32_t bar_full = bar_base;                              // [kStages] used in the leader only
  const uint32_t bar_empty = bar_base + 8 * kStages;               // [kStages] one per CTA
  const uint32_t bar_acc_full = bar_base + 16 * kStages;           // [2] MMA -> epilogue, one per CTA
  const uint32_t bar_acc_free = bar_acc_full + 16;                 // [2] both epilogues -> leader's MMA
  const uint32_t bar_ovl_free = bar_acc_free + 16;                 // [2] likewise, shared columns
  const uint32_t tmem_slot = bar_ovl_free + 16;
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  // (the shuffle tells the compiler that the warp index is the same in all lanes, so that role
  // branches and everything computed under them can use the uniform datapath)
  const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();            // 0 = leader
  const int pair = blockIdx.x >> 1;
  const int num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8 * b, 1);
      mbar_init(bar_acc_free + 8 * b, 8);    // 4 epilogue warps in each of the two CTAs
      mbar_init(bar_ovl_free + 8 * b, 8);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    gemm::tmem_alloc(tmem_slot, kTmemCols);
    gemm::tmem_relinquish();
  }
  gemm::tc_fence_before();
  __syncthreads();
  cluster_sync_all();                       // the partner's barriers exist before anyone signals them
  gemm::tc_fence_after();
  griddep_launch_dependents();
  griddep_wait();                           // operands come from the kernel before; y may still be read by it
  const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, *tmem_slot_ptr, 0);
  const uint32_t tmem_sfa = tmem_base + kSfaCol;
  const uint32_t tmem_sfb = tmem_base + kSfbCol;

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    // All 32 lanes walk the loop together (uniform addresses and counters); lane 0 issues.
    {
      const uint32_t issue = lane == 0 ? 1u : 0u;
      if (lane == 0) {
        tma_prefetch_desc(&tma);
        tma_prefetch_desc(&tmw);
        tma_prefetch_desc(&tmsfa);
        tma_prefetch_desc(&tmsfb);
        if (p.total_units > p.full_units) tma_prefetch_desc(&tmw_half);
      }
      int stage = 0;
      uint32_t phase = 0;
      int64_t issued = 0;
      bool ok = true;
      const uint32_t full0 = map_to_cta(bar_full, 0);      // the leader's barriers, as seen from here
      for (int u = pair; u < p.total_units && ok; u += num_pairs) {
        int tile, half, bn, tm, tn;
        unit_tile(u, p, tile, half, bn);
        tile_coords(tile, p, tm, tn);
        const int m0 = tm * 256 + (int)rank * kBM;
        const int n0 = tn * kBN + half * (kBN / 2);
        // a half-width unit brings half as many W rows per CTA (through the map with the smaller box)
        const uint32_t stage_tx = 2u * (uint32_t)(kStageBytes - (bn == kBN ? 0 : kBTileBytes / 2));
        for (int ks = 0; ks < p.num_k_steps; ++ks) {
          if (issued >= kStages) ok = mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1u, SITE_GEMM_EMPTY);
          if (!ok) break;
          if (rank == 0) mbar_arrive_expect_tx_if(issue, bar_full + 8 * stage, stage_tx);
          const uint32_t full = full0 + 8 * stage;
          tma_load_2d_pair_if(issue, sA + stage * kATileBytes, &tma, ks * 128, m0, full);
          if (bn == kBN)
            tma_load_2d_pair_if(issue, sB + stage * kBTileBytes, &tmw, ks * 128, n0 + (int)rank * (kBN / 2), full);
          else
            tma_load_2d_pair_if(issue, sB + stage * kBTileBytes, &tmw_half, ks * 128, n0 + (int)rank * (kBN / 4), full);
          // scale maps are in 32-bit elements: one K step = 1024 bytes = 256 elements per row block
          tma_load_2d_pair_if(issue, sSFA + stage * kSfaBytes, &tmsfa, ks * 256, m0 >> 7, full);
          tma_load_2d_pair_if(issue, sSFB + stage * kSfbBytes, &tmsfb, ks * 256, n0 >> 7, full);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && rank == 0) {
        // Do not go on to the exit while copies may still land: wait (bounded) for the last load
        // armed on every stage.  The partner's copies are counted on the same barriers.
        const int64_t first = issued > kStages ? issued - kStages : 0;
        for (int64_t i = first; i < issued; ++i)
          mbar_wait_warp(bar_full + 8 * (int)(i % kStages), (uint32_t)((i / kStages) & 1), SITE_GEMM_DRAIN);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) ------------------------------
    // All 32 lanes of the leader's warp walk the loop together; lane 0 issues for the pair.
    if (rank == 0) {
      const gemm::IssueRing ring = {sA, sB, sSFA, sSFB, bar_full, bar_empty, bar_acc_full, bar_acc_free, bar_ovl_free};
      auto units_below = [&](int limit) {   // how many of this pair's units have an index below `limit`
        return pair < limit ? (limit - pair + num_pairs - 1) / num_pairs : 0;
      };
      gemm::mma_issue_loop<2, kBN, kStages, kATileBytes, kBTileBytes, kSfaBytes, kSfbBytes, kAccStride, true>(
          ring, tmem_base, tmem_sfa, tmem_sfb, make_idesc_pair<kBN>(), units_below(p.total_units), p.num_k_steps,
          lane == 0, units_below(p.full_units), make_idesc_pair<kBN / 2>());
    }
  } else {
    // ------------------------------ epilogue (both CTAs) ------------------------------
    const int q = warp & 3;
    int it = 0;
    for (int u = pair; u < p.total_units; u += num_pairs, ++it) {
      int tile, half, bn, tm, tn;
      unit_tile(u, p, tile, half, bn);
      tile_coords(tile, p, tm, tn);
      const int buf = it & 1;
      if (!mbar_wait_warp(bar_acc_full + 8 * buf, (uint32_t)((it >> 1) & 1), SITE_GEMM_ACC_FULL)) break;
      gemm::tc_fence_after();
      const uint32_t ovl_free_leader = map_to_cta(bar_ovl_free + 8 * buf, 0);
      const uint32_t acc_free_leader = map_to_cta(bar_acc_free + 8 * buf, 0);
      const uint32_t tmem_acc = tmem_base + buf * kAccStride + ((uint32_t)(q * 32) << 16);
      const int row0 = tm * 256 + (int)rank * kBM + q * 32;
      const int n0 = tn * kBN + half * (kBN / 2);
      const uint32_t stage_buf = sOut + (uint32_t)q * (32u * 128u);
      auto release_shared = [&] { mbar_arrive_cluster(ovl_free_leader); };
      auto release_all = [&] { mbar_arrive_cluster(acc_free_leader); };
      if (bn == kBN)
        gemm::epilogue_tile<kChunks, true, OUT_F32>(tmem_acc, buf, lane, row0, n0, p.M, p.N, p.y, p.ldy, &tmy, stage_buf,
                                                    0u, release_shared, release_all);
      else
        gemm::epilogue_tile<kChunks / 2, true, OUT_F32>(tmem_acc, buf, lane, row0, n0, p.M, p.N, p.y, p.ldy, &tmy,
                                                        stage_buf, 0u, release_shared, release_all);
    }
    // the staging buffer must have been read before this CTA's shared memory goes away; the writes
    // themselves complete with the kernel
    if (!OUT_F32 && lane == 0) gemm::bulk_wait_read<0>();
  }
  gemm::tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the partner is done with this CTA's shared memory, barriers and TMEM
  if (warp == 1) gemm::tmem_dealloc(tmem_base, kTmemCols);
}

bro_status make_scale_map(CUtensorMap* map, const void* scales, int64_t rows, int64_t kblocks, int box_rows);

// How many CTA pairs can be resident at once (the grid never exceeds that: tiles are handed out
// with a fixed stride, so a pair that starts late would finish late).
template <typename Kern>
inline int max_resident_pairs(Kern kernel, int sm_count) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(sm_count & ~1), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return 0;
  }
  return n < sm_count / 2 ? n : sm_count / 2;
}

inline bro_status launch(const void* acodes, const void* ascales, const void* wcodes, const void* wscales,
                         int64_t M, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype, uint32_t flags,
                         int sm_count, cudaStream_t st) {
  Params p;
  p.y = y;
  p.M = M; p.N = N; p.ldy = ldy;
  p.num_k_steps = (int)((K + kBK - 1) / kBK);
  const int64_t kblocks = 2 * (int64_t)p.num_k_steps;
  p.tiles_m = (int)((M + 255) / 256);
  p.tiles_n = (int)((N + kBN - 1) / kBN);
  const int64_t total = (int64_t)p.tiles_m * p.tiles_n;
  if (total > 0x3FFFFFFF) return BRO_ERR_UNSUPPORTED;
  p.total_tiles = (int)total;
  CUtensorMap tma, tmw, tmw_half, tmsfa, tmsfb, tmy;
  bro_status rc = gemm::make_codes_map(&tma, acodes, M, K, kBM);
  if (rc != BRO_OK) return rc;
  rc = gemm::make_codes_map(&tmw, wcodes, N, K, kBN / 2);
  if (rc != BRO_OK) return rc;
  rc = gemm::make_codes_map(&tmw_half, wcodes, N, K, kBN / 4);
  if (rc != BRO_OK) return rc;
  rc = make_scale_map(&tmsfa, ascales, M, kblocks, 1);
  if (rc != BRO_OK) return rc;
  rc = make_scale_map(&tmsfb, wscales, N, kblocks, 2);
  if (rc != BRO_OK) return rc;
  if (out_dtype == BRO_OUT_BF16) {
    rc = gemm::make_out_map(&tmy, y, M, N, ldy);
    if (rc != BRO_OK) return rc;
  } else {
    tmy = tma;   // unused by the fp32-output kernel
  }
  auto go = [&](void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, Params),
                int which) -> bro_status {
    static DeviceOnce once[2];
    int resident = 0;
    const bro_status rc = device_once(once[which], &resident, [&](int* n) {
      if (!cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes),
                   "cudaFuncSetAttribute(gemm pair)"))
        return BRO_ERR_CUDA;
      *n = max_resident_pairs(kernel, sm_count);
      if (*n <= 0) {
        snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "no resident 2-CTA cluster fits on this device");
        return BRO_ERR_CUDA;
      }
      return BRO_OK;
    });
    if (rc != BRO_OK) return rc;
    // Rounds of the persistent grid: when the last round would leave at least half of the pairs idle,
    // its tiles are cut into two half-width units each (BRO_FLAG_GEMM_NO_SPLIT switches this off).
    const int64_t rem = total % resident;
    const bool split = rem > 0 && 2 * rem <= resident && !(flags & BRO_FLAG_GEMM_NO_SPLIT);
    p.full_units = (int)(split ? total - rem : total);
    p.total_units = (int)(split ? total + rem : total);
    const int64_t pairs = p.total_units < resident ? p.total_units : resident;
    return cuda_ok(launch_kernel(kernel, (unsigned)(2 * pairs), kThreads, kSmemBytes, st, 2, tma, tmw, tmw_half, tmsfa,
                                 tmsfb, tmy, p),
                   "gemm_mxfp4 pair launch")
               ? BRO_OK
               : BRO_ERR_CUDA;
  };
  return out_dtype == BRO_OUT_F32 ? go(gemm_mxfp4_pair_kernel<true>, 1) : go(gemm_mxfp4_pair_kernel<false>, 0);
}

}  // namespace gemm2
}  // namespace bro
