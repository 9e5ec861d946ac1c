// Kernel 2: block-scaled MXFP4 x MXFP4 GEMM on the 5th-generation tensor cores
// (paper Sec. 1 / Sec. 4.2: W4A4, y = Q(xR) Q(WR)^T; fp32 accumulation, bf16 or fp32 output).
//
//   y[m, n] = sum_g 2^(Ea[m,g] + Ew[n,g]) * sum_{k in g} a[m,k] w[n,k]
//
// Persistent kernel, one CTA per SM, 128 x BN output tiles handed out round-robin.
// Warp-specialised, every role loops over the CTA's tiles so that the stages of consecutive
// tiles overlap:
//   warp 0      TMA producer: per 256-element K step, one 128x128-byte box of A codes, one
//               BNx128-byte box of W codes (128-byte swizzle) and the matching 512-byte scale
//               blocks (plain bulk copies; the scale tensors are already in tensor-core order).
//               The shared-memory ring runs ahead across tile boundaries.
//   warp 1      owns TMEM; one elected thread copies the scale blocks shared -> TMEM
//               (tcgen05.cp) and issues four tcgen05.mma kind::mxf4.block_scale (K = 64 each)
//               per K step into one of two fp32 accumulators in TMEM; tcgen05.commit releases the
//               shared-memory stage and, after the last K step, hands the accumulator over.
//   warps 2..5  epilogue, each warp on its own for the 32 rows of its TMEM lane quadrant:
//               tcgen05.ld of 64 columns (the next 64 in flight), convert to bf16, stage in the
//               warp's shared-memory buffer (128-byte swizzle), one TMA store of a 64 x 32 box
//               (which also clips the ragged edges); the fp32 output mode stores from registers.
// TMEM holds 512 columns.  For BN = 256 two full accumulators plus the scale columns do not
// fit, so the two accumulators overlap by 32 columns ([0,256) and [224,480)): the epilogue drains
// the shared 32 columns first and releases them early, and the next tile's MMAs start as soon as
// those columns and the rest of its own buffer are free.
// Every mbarrier wait is bounded; on expiry the role records the site and falls through to the
// common exit, where outstanding copies are awaited and TMEM is released.
#pragma once

#include "bro_common.cuh"

namespace bro {
namespace gemm {

constexpr int kBM = 128;
constexpr int kBK = 256;                    // elements per K step = 128 bytes of codes per row
constexpr int kThreads = 192;
constexpr int kATileBytes = kBM * 128;      // 16 KiB
constexpr int kChunkCols = 32;              // epilogue chunk: 32 fp32 columns per tcgen05.ld
constexpr int kRasterRows = 8;              // tile rows per raster band (12 when the weights do not fit L2, see launch_tile)
constexpr int kStageOutBytes = kBM * kChunkCols * 2;   // 8 KiB bf16 staging per chunk

template <int BN> struct Cfg {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kBTileBytes = BN * 128;
  static constexpr int kSfaBytes = 1024;                  // 2 blocks of 512 B (128 rows x 4 groups)
  static constexpr int kSfbBytes = (BN / 128) * 1024;
  static constexpr int kStageBytes = kATileBytes + kBTileBytes + kSfaBytes + kSfbBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 2 * kStageOutBytes + 1024 /*align*/ + 256 /*barriers*/;
  static constexpr int kTmemCols = 512;
  static constexpr int kAccStride = BN == 256 ? 224 : BN;   // column offset of accumulator 1
  static constexpr bool kOverlap = BN == 256;               // accumulators share 32 columns
  static constexpr int kSfaCol = 480;                       // 8 columns: 2 K-blocks x 4
  static constexpr int kSfbCol = 488;                       // up to 16 columns: 2 K-blocks x BN/32
  static constexpr int kChunks = BN / kChunkCols;
};

struct Params {
  const uint8_t* ascales;
  const uint8_t* wscales;
  void* y;
  int64_t M, N, K, ldy;
  int64_t kblocks;          // 512-byte scale blocks per 128-row block = 2*ceil(K/256)
  int num_k_steps;          // ceil(K/256)
  int tiles_m, tiles_n, total_tiles;
  // Work units: units [0, full_units) are whole 128 x BN tiles in row-major tile order; when the
  // tile count leaves the last round of the grid less than half full, the remaining tiles are cut
  // into two 128 x BN/2 halves each (units full_units ..), so that the last round keeps every SM busy.
  int full_units, total_units;
  int raster_rows;          // tile rows per raster band
  int a_box_bytes;          // bytes one activation TMA box brings (fewer than 128 rows when M is small)
  int w_static;             // the weight operand was complete before the previous kernel started (see launch)
};

// ---- tcgen05 wrappers ------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// ---- issuing tensor-core work --------------------------------------------------------------------
// The issuing warp runs its loop with all 32 lanes converged, so that addresses, descriptors and
// loop counters stay warp-uniform: the tensor-core instructions take their operands from uniform
// registers, and values computed under a divergent branch (or derived from something the compiler
// cannot prove uniform, such as a raw threadIdx or a shared-memory load) have to cross register
// files one by one, which makes instruction issue, not the tensor pipe, the limit.  One lane
// executes the instruction itself: every wrapper below predicates it on `issue` (non-zero in that lane).
// CG = 1: this CTA alone; CG = 2: the CTA pair (cta_group::2), issued by the leader CTA.
template <int CG>
__device__ __forceinline__ void tc_commit(uint32_t issue, uint32_t bar) {
  if constexpr (CG == 1)
    asm volatile(
        "{ .reg .pred q; setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0]; }" ::"r"(bar),
        "r"(issue)
        : "memory");
  else   // arrives on the barrier at this offset in both CTAs of the pair
    asm volatile(
        "{ .reg .pred q; setp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %2; }" ::"r"(bar),
        "r"(issue), "h"((uint16_t)3)
        : "memory");
}
// Descriptors are passed as their two 32-bit halves: the upper half is a constant per descriptor
// kind, the lower half is base + a small offset, so no 64-bit arithmetic is needed per instruction.
template <int CG>
__device__ __forceinline__ void tc_cp_sf(uint32_t issue, uint32_t taddr, uint32_t desc_lo, uint32_t desc_hi) {
  if constexpr (CG == 1)
    asm volatile(
        "{ .reg .pred q; .reg .b64 d; setp.ne.b32 q, %3, 0; mov.b64 d, {%1, %2};\n\t"
        "@q tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], d; }" ::"r"(taddr),
        "r"(desc_lo), "r"(desc_hi), "r"(issue)
        : "memory");
  else
    asm volatile(
        "{ .reg .pred q; .reg .b64 d; setp.ne.b32 q, %3, 0; mov.b64 d, {%1, %2};\n\t"
        "@q tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], d; }" ::"r"(taddr),
        "r"(desc_lo), "r"(desc_hi), "r"(issue)
        : "memory");
}
template <int CG>
__device__ __forceinline__ void tc_mma_mxf4(uint32_t issue, uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo,
                                            uint32_t desc_hi, uint32_t idesc, uint32_t sfa_tmem, uint32_t sfb_tmem,
                                            uint32_t accumulate) {
  if constexpr (CG == 1)
    asm volatile(
        "{ .reg .pred p, q; .reg .b64 da, db; setp.ne.b32 p, %7, 0; setp.ne.b32 q, %8, 0;\n\t"
        "mov.b64 da, {%1, %3}; mov.b64 db, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %4, [%5], [%6], p; }" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate), "r"(issue)
        : "memory");
  else
    asm volatile(
        "{ .reg .pred p, q; .reg .b64 da, db; setp.ne.b32 p, %7, 0; setp.ne.b32 q, %8, 0;\n\t"
        "mov.b64 da, {%1, %3}; mov.b64 db, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], da, db, %4, [%5], [%6], p; }" ::"r"(d_tmem),
        "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(sfa_tmem), "r"(sfb_tmem), "r"(accumulate), "r"(issue)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- descriptors -------------------------------------------------------------------------------
// Shared-memory matrix descriptor, K-major operand stored as rows of 128 bytes with the 128-byte
// swizzle (8-row groups 1024 bytes apart).  Low word: start address / 16 in bits 0..13, leading
// byte offset / 16 = 1 in bits 16..29 (unused with swizzle).  High word: stride byte offset / 16
// in bits 0..13, descriptor version 1 in bit 14, layout 2 (128-byte swizzle) in bits 29..31.
// Advancing by 64 K elements (32 bytes) inside the swizzled row adds 2 to the low word.
constexpr uint32_t kDescHiSw128 = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo_sw128(uint32_t saddr) { return ((saddr >> 4) & 0x3FFFu) | (1u << 16); }
// Scale block: 32 rows x 16 bytes, dense, no swizzle; 8-row groups 128 bytes apart.
constexpr uint32_t kDescHiSf = (128u >> 4) | (1u << 14);
__device__ __forceinline__ uint32_t desc_lo_sf(uint32_t saddr) { return (saddr >> 4) & 0x3FFFu; }
// Instruction descriptor, kind::mxf4 block-scaled: E2M1 x E2M1, both K-major, UE8M0 scales,
// dense K = 64, M x N = 128 x BN; scale-factor byte ids filled in per K block.
template <int BN>
__device__ __forceinline__ constexpr uint32_t make_idesc() {
  return (1u << 7) /*A = E2M1*/ | (1u << 10) /*B = E2M1*/ | ((uint32_t)(BN >> 3) << 17) | (1u << 23) /*UE8M0*/ |
         ((uint32_t)(kBM >> 4) << 24);
}


// Barrier over `nthreads` threads that also ANDs a predicate, so that all of them take the same
// branch afterwards (used to leave the tile loop together after a lost wait).
__device__ __forceinline__ bool named_barrier_and(int id, int nthreads, bool pred) {
  uint32_t out;
  asm volatile(
      "{ .reg .pred p, q; setp.ne.u32 q, %3, 0; bar.red.and.pred p, %1, %2, q; selp.u32 %0, 1, 0, p; }"
      : "=r"(out)
      : "r"(id), "r"(nthreads), "r"((uint32_t)pred)
      : "memory");
  return out != 0;
}
__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// TMA store shared -> global of one box; out-of-range parts of the box are clipped.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(m)),
               "r"(src), "r"(x), "r"(y)
               : "memory");
}
// One-lane forms for a converged warp (`issue` non-zero in the issuing lane; operands uniform).
__device__ __forceinline__ void tma_store_2d_if(uint32_t issue, const CUtensorMap* m, uint32_t src, int x, int y) {
  asm volatile(
      "{ .reg .pred q; setp.ne.b32 q, %4, 0;\n\t"
      "@q cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1]; }" ::"l"(
          reinterpret_cast<uint64_t>(m)),
      "r"(src), "r"(x), "r"(y), "r"(issue)
      : "memory");
}
__device__ __forceinline__ void bulk_commit_if(uint32_t issue) {
  asm volatile("{ .reg .pred q; setp.ne.b32 q, %0, 0;\n\t@q cp.async.bulk.commit_group; }" ::"r"(issue) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read_if(uint32_t issue) {
  asm volatile("{ .reg .pred q; setp.ne.b32 q, %0, 0;\n\t@q cp.async.bulk.wait_group.read %1; }" ::"r"(issue), "n"(N)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Unit index -> first row, first column and width of its output tile.
template <int BN>
__device__ __forceinline__ void decode_unit(const Params& p, int u, int& m0, int& n0, int& bn) {
  int tile = u, half = 0;
  bn = BN;
  if (u >= p.full_units) {
    const int idx = u - p.full_units;
    tile = p.full_units + (idx >> 1);
    half = idx & 1;
    bn = BN / 2;
  }
  // Tile order: bands of raster_rows tile rows, column by column inside a band, so that the CTAs
  // running at the same time share a few activation panels and a few weight panels (with plain
  // row-major order and a weight matrix larger than L2, every tile row streams W from HBM again).
  const int per_band = p.raster_rows * p.tiles_n;
  const int band = tile / per_band;
  const int within = tile - band * per_band;
  const int rows = min(p.raster_rows, p.tiles_m - band * p.raster_rows);
  const int tn = within / rows;
  const int tm = band * p.raster_rows + (within - tn * rows);
  m0 = tm * kBM;
  n0 = tn * BN + half * (BN / 2);
}

// Addresses the issuing warp works with (shared-memory window addresses of stage 0 and of the
// first barrier of each kind).
struct IssueRing {
  uint32_t sA, sB, sSFA, sSFB;
  uint32_t bar_full, bar_empty, bar_acc_full, bar_acc_free, bar_ovl_free;
};

// The K loop of the issuing warp over all tiles of this CTA (or CTA pair), shared by both kernels.
// Per 256-element K step: two scale-block copies shared -> TMEM per operand row block and four
// MMAs of K = 64.  The two 128-element halves of a step own separate TMEM scale columns
// (A: 4 columns at 4h; W: BN/32 columns at (BN/32)h), and the copies for the NEXT step are issued
// between the halves of the current one, so a copy never sits directly in front of its consumer.
// Accumulator t & 1 is used for this CTA's t-th tile; with OVERLAP the two accumulators share
// columns that the epilogue of the other buffer releases through bar_ovl_free.
template <int CG, int BN, int STAGES, int A_STAGE, int B_STAGE, int SFA_STAGE, int SFB_STAGE, int ACC_STRIDE,
          bool OVERLAP>
__device__ __forceinline__ void mma_issue_loop(const IssueRing& r, uint32_t tmem_base, uint32_t tmem_sfa,
                                               uint32_t tmem_sfb, uint32_t idesc_full, int my_tiles, int num_k_steps,
                                               bool issue_lane, int narrow_from = 0x7FFFFFFF,
                                               uint32_t idesc_narrow = 0u) {
  // tiles narrow_from.. of this CTA are half-width: same loop, the instruction descriptor says N = BN/2
  const uint32_t issue = issue_lane ? 1u : 0u;
  const uint32_t a_lo0 = desc_lo_sw128(r.sA), b_lo0 = desc_lo_sw128(r.sB);
  const uint32_t sfa_lo0 = desc_lo_sf(r.sSFA), sfb_lo0 = desc_lo_sf(r.sSFB);
  const uint32_t hi_op = kDescHiSw128, hi_sf = kDescHiSf;
  uint32_t idesc0 = idesc_full;
  // scale bytes {0,1} of a 32-bit scale word for the first MMA of a half, {2,3} for the second
  uint32_t idesc1 = idesc0 | (2u << 4) | (2u << 29);
  // (a half-width unit reads the scales of its one 128-row block of W only)
  auto copy_scales = [&](int stage, int h, bool narrow) {
    const uint32_t lo_a = sfa_lo0 + (uint32_t)stage * (SFA_STAGE >> 4) + (uint32_t)h * 32u;
    const uint32_t lo_b = sfb_lo0 + (uint32_t)stage * (SFB_STAGE >> 4) + (uint32_t)h * 32u;
    tc_cp_sf<CG>(issue, tmem_sfa + 4 * h, lo_a, hi_sf);
    tc_cp_sf<CG>(issue, tmem_sfb + (BN / 32) * h, lo_b, hi_sf);
    if (BN == 256 && !narrow) tc_cp_sf<CG>(issue, tmem_sfb + (BN / 32) * h + 4, lo_b + 64u, hi_sf);
  };
  auto mma_half = [&](int stage, int h, uint32_t tmem_acc, uint32_t accumulate_first) {
    const uint32_t a_lo = a_lo0 + (uint32_t)stage * (A_STAGE >> 4) + 4u * h;
    const uint32_t b_lo = b_lo0 + (uint32_t)stage * (B_STAGE >> 4) + 4u * h;
    const uint32_t tsfa = tmem_sfa + 4 * h, tsfb = tmem_sfb + (BN / 32) * h;
    tc_mma_mxf4<CG>(issue, tmem_acc, a_lo, b_lo, hi_op, idesc0, tsfa, tsfb, accumulate_first);
    tc_mma_mxf4<CG>(issue, tmem_acc, a_lo + 2u, b_lo + 2u, hi_op, idesc1, tsfa | (2u << 30), tsfb | (2u << 30), 1u);
  };
  int stage = 0;
  uint32_t phase = 0;
  bool ok = my_tiles > 0;
  if (ok) ok = mbar_wait_warp(r.bar_full, 0u, SITE_GEMM_FULL);
  if (ok) {
    tc_fence_after();
    copy_scales(0, 0, 0 >= narrow_from);
    copy_scales(0, 1, 0 >= narrow_from);
  }
  for (int it = 0; it < my_tiles && ok; ++it) {
    const int buf = it & 1;
    const int use = it >> 1;                       // how many times this buffer was used before
    // this buffer must have been drained by the epilogue of tile it-2 ...
    if (use >= 1) ok = mbar_wait_warp(r.bar_acc_free + 8 * buf, (uint32_t)((use - 1) & 1), SITE_GEMM_ACC_EMPTY);
    // ... and the columns it shares with the other buffer by the epilogue of tile it-1
    if (ok && OVERLAP && it >= 1)
      ok = mbar_wait_warp(r.bar_ovl_free + 8 * (buf ^ 1), (uint32_t)(((it - 1) >> 1) & 1), SITE_GEMM_ACC_EMPTY);
    if (!ok) break;
    tc_fence_after();
    const uint32_t tmem_acc = tmem_base + buf * ACC_STRIDE;
    if (it >= narrow_from) {
      idesc0 = idesc_narrow;
      idesc1 = idesc0 | (2u << 4) | (2u << 29);
    }
    for (int ks = 0; ks < num_k_steps; ++ks) {
      const bool has_next = (ks + 1 < num_k_steps) || (it + 1 < my_tiles);
      const int next_stage = (stage + 1 == STAGES) ? 0 : stage + 1;
      const uint32_t next_phase = (stage + 1 == STAGES) ? (phase ^ 1u) : phase;
      const bool next_narrow = (ks + 1 < num_k_steps ? it : it + 1) >= narrow_from;   // the unit the next stage belongs to
      // Probe the next stage's barrier before issuing: the answer travels while the two MMAs
      // below are issued, and in the steady state it is "ready", so the issuing warp rarely
      // spends a barrier round trip between tensor-core instructions.
      const bool probe = has_next && mbar_try_wait(r.bar_full + 8 * next_stage, next_phase);
      mma_half(stage, 0, tmem_acc, ks == 0 ? 0u : 1u);
      if (has_next) {
        if (!__all_sync(0xFFFFFFFFu, probe)) ok = mbar_wait_warp(r.bar_full + 8 * next_stage, next_phase, SITE_GEMM_FULL);
        if (!ok) break;
        tc_fence_after();
        copy_scales(next_stage, 0, next_narrow);   // half 0's columns were last read by the two MMAs above
      }
      mma_half(stage, 1, tmem_acc, 1u);
      tc_commit<CG>(issue, r.bar_empty + 8 * stage);   // frees the stage when these MMAs have read it
      if (has_next) copy_scales(next_stage, 1, next_narrow);
      stage = next_stage;
      phase = next_phase;
    }
    tc_commit<CG>(issue, r.bar_acc_full + 8 * buf);    // accumulator complete (or abandoned) -> epilogue
  }
}

// One epilogue warp's share of one finished accumulator: the 32 rows of its TMEM lane quadrant,
// CHUNKS chunks of 32 columns, handled two chunks (64 columns) at a time.  The warp works on its
// own — no barrier between warps: tcgen05.ld of the next pair is in flight while the current one is
// converted to bf16, written to the warp's staging buffer (32 rows x 128 bytes, 128-byte swizzle)
// and sent off with ONE TMA store of a 64 x 32 box, which clips rows beyond M and columns beyond N.
// (Tried and slower: st.global straight from registers, and a transpose through shared memory
// followed by coalesced 16-byte st.global — both make the whole kernel 15-20 % slower on
// output-heavy shapes; the asynchronous TMA store is what keeps the epilogue off the critical path.)
// Pair order: the pair that holds the columns shared with the other accumulator first (buffer 0
// shares its last chunk, buffer 1 its first); `release_shared` / `release_all` are called once
// those columns / all columns have been read into registers.
template <int CHUNKS, bool OVERLAP, bool OUT_F32, typename ReleaseShared, typename ReleaseAll>
__device__ __forceinline__ void epilogue_tile(uint32_t tmem_acc, int buf, int lane, int row0, int n0, int64_t M,
                                              int64_t N, void* y, int64_t ldy, const CUtensorMap* tmy,
                                              uint32_t stage_buf, uint32_t stage_stride,
                                              ReleaseShared release_shared, ReleaseAll release_all) {
  // stage_stride == 0: one staging buffer, reused pair after pair (each reuse waits until the
  // previous TMA store has read it).  stage_stride != 0: pair i has its own buffer at
  // stage_buf + i * stage_stride and nothing waits — used for a CTA's final tile, whose epilogue
  // is the kernel's tail and for which the idle operand stages provide the room.
  static_assert(CHUNKS % 2 == 0, "chunks are processed in pairs");
  constexpr int PAIRS = CHUNKS / 2;
  const int64_t row = (int64_t)row0 + lane;
  const uint32_t issue = lane == 0 ? 1u : 0u;
  auto pair_of = [&](int pi) { return (OVERLAP && buf == 0) ? (pi == 0 ? PAIRS - 1 : pi - 1) : pi; };
  auto released = [&](int pi) {
    if (pi == 0 || pi == PAIRS - 1) {
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (pi == 0) release_shared();
        if (pi == PAIRS - 1) release_all();
      }
    }
  };
  auto store_f32 = [&](const uint32_t (&r)[32], int col0) {
    if (row < M && col0 < N) {
      float* dst = static_cast<float*>(y) + row * ldy + col0;
      if ((int64_t)col0 + 32 <= N) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
          reinterpret_cast<uint4*>(dst)[j] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
      } else {
        for (int j = 0; j < 32 && col0 + j < N; ++j) dst[j] = __uint_as_float(r[j]);
      }
    }
  };
  auto emit = [&](const uint32_t (&r0)[32], const uint32_t (&r1)[32], int pr, int pi) {
    const int col0 = n0 + pr * 2 * kChunkCols;
    if (OUT_F32) {
      store_f32(r0, col0);
      store_f32(r1, col0 + kChunkCols);
    } else {
      uint32_t h[32];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(h[j]) : "f"(__uint_as_float(r0[2 * j + 1])), "f"(__uint_as_float(r0[2 * j])));
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(h[16 + j]) : "f"(__uint_as_float(r1[2 * j + 1])), "f"(__uint_as_float(r1[2 * j])));
      }
      const uint32_t sbuf = stage_buf + (uint32_t)pi * stage_stride;
      // the TMA store that last read the staging buffer must be done reading it
      if (stage_stride == 0u) bulk_wait_read_if<0>(issue);
      __syncwarp();
      // row `lane` of the box: 128 bytes, 16-byte pieces XOR-swizzled with lane & 7
      const uint32_t rowaddr = sbuf + (uint32_t)lane * 128u;
      const uint32_t sw = (uint32_t)lane & 7u;
#pragma unroll
      for (int j = 0; j < 8; ++j) sts128(rowaddr + ((j ^ sw) << 4), h[4 * j], h[4 * j + 1], h[4 * j + 2], h[4 * j + 3]);
      fence_proxy_async_smem();
      __syncwarp();
      // A TMA store clips at 16-byte granularity: when N is not a multiple of 8 the ragged last
      // pair is written from registers instead, element by element.
      const bool ragged = ((N & 7) != 0) && ((int64_t)col0 + 2 * kChunkCols > N);
      tma_store_2d_if((col0 < N && row0 < M && !ragged) ? issue : 0u, tmy, sbuf, col0, row0);
      bulk_commit_if(issue);           // (possibly empty) keeps the group count in step
      if (ragged && row < M) {
        uint16_t* dst = static_cast<uint16_t*>(y) + row * ldy + col0;
#pragma unroll
        for (int j = 0; j < 64; ++j)
          if ((int64_t)col0 + j < N) dst[j] = (uint16_t)((j & 1) ? (h[j >> 1] >> 16) : (h[j >> 1] & 0xFFFFu));
      }
    }
  };
  uint32_t ra[32], rb[32], rc[32], rd[32];
  tc_ld32(tmem_acc + pair_of(0) * 2 * kChunkCols, ra);
  tc_ld32(tmem_acc + pair_of(0) * 2 * kChunkCols + kChunkCols, rb);
#pragma unroll
  for (int pi = 0; pi < PAIRS; pi += 2) {
    tc_wait_ld();
    if (pi + 1 < PAIRS) {
      tc_ld32(tmem_acc + pair_of(pi + 1) * 2 * kChunkCols, rc);
      tc_ld32(tmem_acc + pair_of(pi + 1) * 2 * kChunkCols + kChunkCols, rd);
    }
    released(pi);
    emit(ra, rb, pair_of(pi), pi);
    if (pi + 1 < PAIRS) {
      tc_wait_ld();
      if (pi + 2 < PAIRS) {
        tc_ld32(tmem_acc + pair_of(pi + 2) * 2 * kChunkCols, ra);
        tc_ld32(tmem_acc + pair_of(pi + 2) * 2 * kChunkCols + kChunkCols, rb);
      }
      released(pi + 1);
      emit(rc, rd, pair_of(pi + 1), pi + 1);
    }
  }
}

template <int BN, bool OUT_F32>
__global__ void __launch_bounds__(kThreads, 1)
gemm_mxfp4_kernel(const __grid_constant__ CUtensorMap tma, const __grid_constant__ CUtensorMap tmw,
                  const __grid_constant__ CUtensorMap tmw_half, const __grid_constant__ CUtensorMap tmy,
                  const Params p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sA = smem_base;
  const uint32_t sB = sA + C::kStages * kATileBytes;
  const uint32_t sSFA = sB + C::kStages * C::kBTileBytes;
  const uint32_t sSFB = sSFA + C::kStages * C::kSfaBytes;
  const uint32_t sOut = sSFB + C::kStages * C::kSfbBytes;          // 2 x 8 KiB, 1 KiB aligned
  const uint32_t bar_base = sOut + 2 * kStageOutBytes;
  const uint32_t bar_full = bar_base;                              // [kStages]
  const uint32_t bar_empty = bar_base + 8 * C::kStages;            // [kStages]
  const uint32_t bar_acc_full = bar_base + 16 * C::kStages;        // [2] MMA -> epilogue
  const uint32_t bar_acc_free = bar_acc_full + 16;                 // [2] epilogue -> MMA, whole buffer
  const uint32_t bar_ovl_free = bar_acc_free + 16;                 // [2] epilogue -> MMA, shared columns
  const uint32_t tmem_slot = bar_ovl_free + 16;                    // u32 written by tcgen05.alloc
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  // (the shuffle tells the compiler that the warp index is the same in all lanes, so that role
  // branches and everything computed under them can use the uniform datapath)
  const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full + 8 * b, 1);
      mbar_init(bar_acc_free + 8 * b, 4);    // one arrival per epilogue warp
      mbar_init(bar_ovl_free + 8 * b, 4);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, C::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  griddep_launch_dependents();
  // Operands come from the kernel before, and y may still be read by it — except that in the
  // whole-layer call the packed weights are older than that kernel, so the producer may start
  // fetching the weight half of its first stages while the activations are still being written.
  const bool early_w = p.w_static != 0 && warp == 0;
  if (!early_w) griddep_wait();
  const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, *tmem_slot_ptr, 0);
  const uint32_t tmem_sfa = tmem_base + C::kSfaCol;
  const uint32_t tmem_sfb = tmem_base + C::kSfbCol;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tma);
      tma_prefetch_desc(&tmw);
      if (p.total_units > p.full_units) tma_prefetch_desc(&tmw_half);
      int stage = 0;
      uint32_t phase = 0;
      int64_t issued = 0;
      bool ok = true;
      // loads of one K step of one unit; `part` selects the weight side (1), the activation side (2) or both (3)
      auto issue_step = [&](int m0, int n0, int bn, int ks, int st, int part) {
        // 128-row blocks of W scales that exist for this unit (a half-width unit of a ragged last
        // tile can lie entirely beyond N: no block is read then, its columns are never stored)
        const int nblk_valid = (int64_t)n0 >= p.N ? 0 : ((bn == 256 && (int64_t)n0 + 128 < p.N) ? 2 : 1);
        const uint32_t full = bar_full + 8 * st;
        if (part & 1) {
          mbar_arrive_expect_tx(full, p.a_box_bytes + bn * 128 + C::kSfaBytes + nblk_valid * 1024);
          tma_load_2d(sB + st * C::kBTileBytes, bn == BN ? &tmw : &tmw_half, ks * 128, n0, full);
          const uint8_t* sfb_src = p.wscales + (int64_t)(n0 / 128) * p.kblocks * 512;
          for (int nb = 0; nb < nblk_valid; ++nb)
            bulk_load_1d(sSFB + st * C::kSfbBytes + nb * 1024, sfb_src + ((int64_t)nb * p.kblocks + 2 * ks) * 512, 1024,
                         full);
        }
        if (part & 2) {
          tma_load_2d(sA + st * kATileBytes, &tma, ks * 128, m0, full);
          bulk_load_1d(sSFA + st * C::kSfaBytes, p.ascales + ((int64_t)(m0 / kBM) * p.kblocks + 2 * ks) * 512, 1024, full);
        }
      };
      int pre = 0;                  // K steps of the first unit whose loads are issued here
      if (early_w) {
        if ((int)blockIdx.x < p.total_units) {
          int m0, n0, bn;
          decode_unit<BN>(p, (int)blockIdx.x, m0, n0, bn);
          pre = p.num_k_steps < C::kStages ? p.num_k_steps : C::kStages;
          for (int ks = 0; ks < pre; ++ks) issue_step(m0, n0, bn, ks, ks, 1);   // weights: before the wait
          griddep_wait();
          for (int ks = 0; ks < pre; ++ks) issue_step(m0, n0, bn, ks, ks, 2);   // activations: after it
          issued = pre;
          if (pre == C::kStages) phase = 1u; else stage = pre;
        } else {
          griddep_wait();
        }
      }
      for (int u = blockIdx.x; u < p.total_units && ok; u += gridDim.x) {
        int m0, n0, bn;
        decode_unit<BN>(p, u, m0, n0, bn);
        for (int ks = (u == (int)blockIdx.x ? pre : 0); ks < p.num_k_steps; ++ks) {
          if (issued >= C::kStages) ok = mbar_wait(bar_empty + 8 * stage, phase ^ 1u, SITE_GEMM_EMPTY);
          if (!ok) break;
          issue_step(m0, n0, bn, ks, stage, 3);
          ++issued;
          if (++stage == C::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Do not leave while copies may still land in this CTA's shared memory: wait (bounded)
        // for the last load armed on every stage.
        const int64_t first = issued > C::kStages ? issued - C::kStages : 0;
        for (int64_t i = first; i < issued; ++i)
          mbar_wait(bar_full + 8 * (int)(i % C::kStages), (uint32_t)((i / C::kStages) & 1), SITE_GEMM_DRAIN);
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    const IssueRing ring = {sA, sB, sSFA, sSFB, bar_full, bar_empty, bar_acc_full, bar_acc_free, bar_ovl_free};
    auto units_below = [&](int limit) {   // how many of this CTA's units have an index below `limit`
      return (int)blockIdx.x < limit ? (limit - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    };
    mma_issue_loop<1, BN, C::kStages, kATileBytes, C::kBTileBytes, C::kSfaBytes, C::kSfbBytes, C::kAccStride,
                   C::kOverlap>(ring, tmem_base, tmem_sfa, tmem_sfb, make_idesc<BN>(), units_below(p.total_units),
                                p.num_k_steps, lane == 0, units_below(p.full_units), make_idesc<BN / 2>());
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                 // TMEM lane quadrant this warp may read
    int it = 0;
    for (int u = blockIdx.x; u < p.total_units; u += gridDim.x, ++it) {
      int m0, n0, bn;
      decode_unit<BN>(p, u, m0, n0, bn);
      const int buf = it & 1;
      if (!mbar_wait_warp(bar_acc_full + 8 * buf, (uint32_t)((it >> 1) & 1), SITE_GEMM_ACC_FULL)) break;
      tc_fence_after();
      const uint32_t tmem_acc = tmem_base + buf * C::kAccStride + ((uint32_t)(q * 32) << 16);
      // the final tile of this CTA stages every pair in its own 4 KiB of the (now idle) A stages
      const bool last = u + (int)gridDim.x >= p.total_units;
      const uint32_t stage_buf = last ? sA + (uint32_t)q * (4u * 4096u) : sOut + (uint32_t)q * (32u * 128u);
      const uint32_t stage_stride = last ? 4096u : 0u;
      auto release_shared = [&] { mbar_arrive(bar_ovl_free + 8 * buf); };
      auto release_all = [&] { mbar_arrive(bar_acc_free + 8 * buf); };
      if (bn == BN)
        epilogue_tile<C::kChunks, C::kOverlap, OUT_F32>(tmem_acc, buf, lane, m0 + q * 32, n0, p.M, p.N, p.y, p.ldy, &tmy,
                                                        stage_buf, stage_stride, release_shared, release_all);
      else
        epilogue_tile<C::kChunks / 2, C::kOverlap, OUT_F32>(tmem_acc, buf, lane, m0 + q * 32, n0, p.M, p.N, p.y, p.ldy,
                                                            &tmy, stage_buf, stage_stride, release_shared, release_all);
    }
    // the staging buffer must have been read before this CTA's shared memory goes away; the writes
    // themselves complete with the kernel
    if (!OUT_F32 && lane == 0) bulk_wait_read<0>();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

inline size_t workspace_bytes(int64_t, int64_t, int64_t) { return 0; }

bro_status make_codes_map(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int box_rows);
bro_status make_out_map(CUtensorMap* map, const void* y, int64_t M, int64_t N, int64_t ldy);

template <int BN>
bro_status launch_tile(const CUtensorMap& tma, const CUtensorMap& tmw, const CUtensorMap& tmw_half,
                       const CUtensorMap& tmy, Params& p, int out_dtype, uint32_t flags, int sm_count, cudaStream_t st) {
  using C = Cfg<BN>;
  p.tiles_m = (int)((p.M + kBM - 1) / kBM);
  p.tiles_n = (int)((p.N + BN - 1) / BN);
  const int64_t total = (int64_t)p.tiles_m * p.tiles_n;
  if (total > 0x3FFFFFFF) return BRO_ERR_UNSUPPORTED;
  p.total_tiles = (int)total;
  // One wave of CTAs covers raster_rows activation panels and sm_count / raster_rows weight panels.
  // 8 rows is best while the packed weights stay in L2 between bands; when they do not (measured
  // with 125 MB of weights: 2.7 % faster at M = 32768), the squarer 12 x 12 wave re-reads fewer
  // weight bytes from HBM.
  p.raster_rows = (double)p.N * (double)p.K * (17.0 / 32.0) > 64.0 * 1024 * 1024 ? 12 : kRasterRows;
  // Rounds of the persistent grid: when the last round would leave at least half of the SMs idle,
  // its tiles are cut into two half-width units each (BRO_FLAG_GEMM_NO_SPLIT switches this off).
  int64_t grid = total < sm_count ? total : sm_count;
  const int64_t rem = total % sm_count;
  const bool split = BN == 256 && rem > 0 && 2 * rem <= sm_count && !(flags & BRO_FLAG_GEMM_NO_SPLIT);
  p.full_units = (int)(split ? total - rem : total);
  p.total_units = (int)(split ? total + rem : total);
  if (split && p.total_units < sm_count) grid = p.total_units;
  auto go = [&](void (*kernel)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, Params), int which) -> bro_status {
    static DeviceOnce once[2];      // (per BN through the template, per output type through `which`)
    const bro_status rc = device_once(once[which], nullptr, [&](int*) {
      return cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes),
                     "cudaFuncSetAttribute(gemm)")
                 ? BRO_OK
                 : BRO_ERR_CUDA;
    });
    if (rc != BRO_OK) return rc;
    return cuda_ok(launch_kernel(kernel, (unsigned)grid, kThreads, C::kSmemBytes, st, 1, tma, tmw, tmw_half, tmy, p),
                   "gemm_mxfp4 launch")
               ? BRO_OK
               : BRO_ERR_CUDA;
  };
  return out_dtype == BRO_OUT_F32 ? go(gemm_mxfp4_kernel<BN, true>, 1) : go(gemm_mxfp4_kernel<BN, false>, 0);
}

// w_static: the caller guarantees that wcodes / wscales were complete before the kernel that
// precedes this launch in the stream began (true inside the whole-layer calls, where that kernel is
// the library's own rotate+quantize and signals its dependents only after its own wait).
inline bro_status launch(const void* acodes, const void* ascales, const void* wcodes, const void* wscales,
                         int64_t M, int64_t N, int64_t K, void* y, int64_t ldy, int out_dtype, void* /*ws*/,
                         size_t /*ws_bytes*/, uint32_t flags, int sm_count, cudaStream_t st, bool w_static = false) {
  int bn = N <= 128 ? 128 : 256;
  if (flags & BRO_FLAG_GEMM_TILE_N128) bn = 128;
  else if (flags & BRO_FLAG_GEMM_TILE_N256) bn = 256;
  Params p;
  p.ascales = static_cast<const uint8_t*>(ascales);
  p.wscales = static_cast<const uint8_t*>(wscales);
  p.y = y;
  p.M = M; p.N = N; p.K = K; p.ldy = ldy;
  p.num_k_steps = (int)((K + kBK - 1) / kBK);
  p.kblocks = 2 * (int64_t)p.num_k_steps;
  p.w_static = w_static ? 1 : 0;
  CUtensorMap tma, tmw, tmy;
  // With fewer than 128 tokens the activation box covers only the next power of two of rows (at
  // least 8): rows the box does not bring keep whatever the shared-memory stage held — finite fp4
  // codes under zero-padded scales — and feed output rows that are never stored.
  int a_rows = kBM;
  while (a_rows > 8 && a_rows / 2 >= M) a_rows /= 2;
  p.a_box_bytes = a_rows * 128;
  bro_status rc = make_codes_map(&tma, acodes, M, K, a_rows);
  if (rc != BRO_OK) return rc;
  rc = make_codes_map(&tmw, wcodes, N, K, bn);
  if (rc != BRO_OK) return rc;
  if (out_dtype == BRO_OUT_BF16) {
    rc = make_out_map(&tmy, y, M, N, ldy);
    if (rc != BRO_OK) return rc;
  } else {
    tmy = tma;   // unused by the fp32-output kernel
  }
  CUtensorMap tmw_half;       // the same weights seen through a box of half as many rows
  rc = make_codes_map(&tmw_half, wcodes, N, K, bn / 2);
  if (rc != BRO_OK) return rc;
  return bn == 256 ? launch_tile<256>(tma, tmw, tmw_half, tmy, p, out_dtype, flags, sm_count, st)
                   : launch_tile<128>(tma, tmw, tmw_half, tmy, p, out_dtype, flags, sm_count, st);
}

}  // namespace gemm
}  // namespace bro
