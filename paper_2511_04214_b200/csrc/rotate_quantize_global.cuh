// Kernel 1g: rotation block = K (the global rotation the paper compares against, Sec. 4.2-4.3,
// Sec. 5.2) fused with MXFP4 quantisation.  K = 2^p, 32 <= K <= 32768.
//
// Same arithmetic contract as the block kernel: butterflies with ascending stride in fp32, one
// multiply by fp32(1/sqrt(K)), then per-32 quantisation.  A thread owns one MX group:
//   strides 1..16      in registers,
//   strides 32..512    between lanes (one shuffle per element per stage),
//   strides >= 1024    between warps through shared memory (swizzled, conflict-free float4).
// The global rotation costs log2(K) stages instead of 5; it is expected to run below the HBM
// roofline — that cost difference is the paper's point (Sec. 4.3 "Reduced online computing").
#pragma once

#include "bro_common.cuh"
#include "rotate_quantize.cuh"
#include "fake_quantize.cuh"

namespace bro {
namespace rqg {

struct Params {
  const uint16_t* x;
  int64_t M, K, ldx;
  uint8_t* codes;
  uint8_t* scales;
  int64_t scale_kblocks;
  int layout;
  int log2k;
  int threads_per_row;   // K / 32
  int rows_per_iter;     // blockDim.x / threads_per_row
  const uint16_t* signs; // [K] bf16 +-1 for the randomised rotation diag(s) H / sqrt(K), or nullptr
  float* mse;            // if set: write the per-group quantisation error [M, K/32] instead of codes/scales
  int format;            // ... for this 4-bit format (see rq::group_error)
  float* deq;            // if set: write the dequantised values [M, K] (row stride ldd) under `format` instead
  int64_t ldd;
  uint32_t* rowstats;    // per-row formats: the row ranges (fq::group_range); written when `range_pass` is set
  int range_pass;
};

template <int kMaxThreads>
__global__ void __launch_bounds__(kMaxThreads, 1) rotate_quantize_global_kernel(const Params p) {
  extern __shared__ float xch[];   // [rows_per_iter][K] fp32, only used when K > 1024
  const int T = p.threads_per_row;
  const int gi = threadIdx.x % T;          // group index within the row
  const int rs = threadIdx.x / T;          // row slot within this iteration
  const uint32_t cbits = (p.log2k % 2 == 0) ? (uint32_t)(127 - p.log2k / 2) << 23
                                            : 0x3FB504F3u - ((uint32_t)((p.log2k + 1) / 2) << 23);
  const int64_t row_iters = (p.M + p.rows_per_iter - 1) / p.rows_per_iter;
  griddep_wait();               // x may be written, codes/scales still read, by the kernel before
  // (only now: a dependent that starts early may then rely on everything older than this kernel)
  griddep_launch_dependents();
  // a thread always works on the same 32 channels, so its slice of the sign vector is loaded once
  uint4 sg[4] = {};
  if (p.signs) {
    const uint4* sp = reinterpret_cast<const uint4*>(p.signs + (int64_t)gi * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) sg[j] = __ldg(sp + j);
  }

  for (int64_t it = blockIdx.x; it < row_iters; it += gridDim.x) {
    const int64_t row = it * p.rows_per_iter + rs;
    const bool live = row < p.M;
    uint64_t P[16];
    {
      const uint4* src = reinterpret_cast<const uint4*>(p.x + (live ? row : 0) * p.ldx + (int64_t)gi * 32);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint4 q = live ? __ldg(src + j) : make_uint4(0u, 0u, 0u, 0u);
        rq::unpack_stage1(rq::apply_signs(q, sg[j]), P + 4 * j);
      }
    }
    rq::fwht32_stages_2_to_16(P);
    // lane stages: stride 32 * m, m = 1..16 (only those below K)
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
      if (m < T) rq::cross_lane_stage(P, m, (gi & m) != 0);
    }
    // warp stages through shared memory
    for (int m = 32; m < T; m <<= 1) {
      float* mine = xch + (size_t)rs * p.K + (size_t)gi * 32;
      __syncthreads();   // previous round's reads are done
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        float a0, a1, a2, a3;
        rq::unpack2(P[2 * c], a0, a1);
        rq::unpack2(P[2 * c + 1], a2, a3);
        *reinterpret_cast<float4*>(mine + ((c ^ (gi & 7)) << 2)) = make_float4(a0, a1, a2, a3);
      }
      __syncthreads();
      const int pg = gi ^ m;
      const float* theirs = xch + (size_t)rs * p.K + (size_t)pg * 32;
      const float sgn = (gi & m) ? -1.f : 1.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const float4 o = *reinterpret_cast<const float4*>(theirs + ((c ^ (pg & 7)) << 2));
        float a0, a1, a2, a3;
        rq::unpack2(P[2 * c], a0, a1);
        rq::unpack2(P[2 * c + 1], a2, a3);
        P[2 * c] = rq::pack2(__fmaf_rn(a0, sgn, o.x), __fmaf_rn(a1, sgn, o.y));
        P[2 * c + 1] = rq::pack2(__fmaf_rn(a2, sgn, o.z), __fmaf_rn(a3, sgn, o.w));
      }
    }
    if (p.format == rq::kFormatScaleOnly && !p.deq && !p.range_pass) {   // analysis mode (uniform over the grid): scale byte only
      const uint32_t sbyte = rq::group_scale_byte(P, cbits);
      if (live) p.scales[row * (p.K >> 5) + gi] = (uint8_t)sbyte;
      continue;
    }
    if (p.mse) {                 // analysis mode (uniform over the grid)
      const float e = rq::group_error(P, cbits, p.format);
      if (live) p.mse[row * (p.K >> 5) + gi] = e;
      continue;
    }
    if (p.range_pass) {          // first pass of the per-row formats (uniform over the grid)
      float neglo, hi;
      fq::group_range(P, cbits, neglo, hi);
      if (live) {
        atomicMax(p.rowstats + 2 * row, __float_as_uint(neglo));
        atomicMax(p.rowstats + 2 * row + 1, __float_as_uint(hi));
      }
      continue;
    }
    if (p.deq) {                 // simulated quantisation (uniform over the grid)
      float out[32];
      if (p.format == fq::kFormatNone) {
        const uint64_t cc = rq::pack2(__uint_as_float(cbits), __uint_as_float(cbits));
#pragma unroll
        for (int k = 0; k < 16; ++k) rq::unpack2(rq::mul2(P[k], cc), out[2 * k], out[2 * k + 1]);
      } else if (p.format >= fq::kFormatRowSym) {
        const int64_t r = live ? row : 0;
        fq::row_dequant(P, cbits, p.format == fq::kFormatRowAsym, __uint_as_float(__ldcg(p.rowstats + 2 * r)),
                        __uint_as_float(__ldcg(p.rowstats + 2 * r + 1)), out);
      } else
      fq::group_dequant(P, cbits, p.format, out);
      if (live) fq::store_group(p.deq + row * p.ldd + (int64_t)gi * 32, out);
      continue;
    }
    uint32_t w[4];
    const uint32_t s = rq::quantize_group(P, cbits, w);
    if (live) {
      *reinterpret_cast<uint4*>(p.codes + row * (p.K >> 1) + (int64_t)gi * 16) =
          make_uint4(w[0], w[1], w[2], w[3]);
      if (p.layout == BRO_LAYOUT_GEMM) {
        const int64_t off = ((row >> 7) * p.scale_kblocks + (gi >> 2)) * 512 + (row & 31) * 16 +
                            ((row & 127) >> 5) * 4 + (gi & 3);
        p.scales[off] = (uint8_t)s;
      } else {
        p.scales[row * (p.K >> 5) + gi] = (uint8_t)s;
      }
    }
  }
}

// ---- K = 2048 / 4096, codes path: the stages above stride 16 through two shared-memory transposes ----
// A thread always works on 32 values in registers, but on a different set in each of three phases, so
// that every butterfly stage is register arithmetic (no shuffle in the transform):
//   phase 1   element bits 0..4  : the thread's 32 consecutive channels (as loaded)
//   phase 2   element bits 5..9  : 32 channels 32 apart (one column of a 32 x 32 block)
//   phase 3   element bits 10..  : 2 (K = 2048) or 4 (K = 4096) runs of 16 / 8 consecutive channels, 1024 apart
// Stage order is still ascending stride with one fp32 rounding per add / subtract, so the result is the
// same bit for bit.  Between the phases the row passes through shared memory (fp32, K values per row,
// two buffers so that one barrier per transpose suffices); all accesses are bank-conflict free:
//   transpose 1  writes 8 x 16 bytes per thread, 16-byte pieces XOR-swizzled with the thread index, and
//                reads 32 scalars per thread (a warp reads one 128-byte line per instruction);
//   transpose 2  writes 32 scalars per thread (a warp writes one line per instruction) and reads 8 x 16
//                bytes, pieces swizzled with bits 3..4 of the piece index.
// After phase 3 a thread holds 8 (16) consecutive values of 4 (2) MX groups; the group maximum takes two
// (one) shuffles per group, codes go out as one 32-bit (64-bit) store per group.
// The bf16 rows arrive by TMA (one 8 KiB box per pass: ROWS rows x K/64 segments of 128 bytes, 128-byte
// swizzle), issued by thread 0 for the NEXT pass as soon as every thread has taken its 64 bytes of the
// current one: the load/store unit's data path, which bounds this kernel, then carries only the
// conflict-free shared-memory reads instead of one 128-byte line per two lanes of a global load.
template <int LOG2K, bool SIGNS>
__global__ void __launch_bounds__(128, 5) rotate_quantize_global_smem_kernel(const __grid_constant__ CUtensorMap tmx,
                                                                              const Params p) {
  static_assert(LOG2K == 11 || LOG2K == 12, "K = 2048 or 4096");
  constexpr int K = 1 << LOG2K;
  constexpr int T = K / 32;                   // threads per row
  constexpr int ROWS = 128 / T;               // rows per pass of the CTA
  constexpr int HB = LOG2K - 10;              // element bits handled in phase 3
  constexpr int NJ = 1 << HB;                 // runs per thread in phase 3
  constexpr int RUN = 32 / NJ;                // consecutive values per run
  constexpr uint32_t kRawBytes = (uint32_t)ROWS * K * 2;          // 8 KiB
  extern __shared__ uint8_t smem_raw[];       // [raw bf16 box | barrier | fp32 [2][ROWS][K]], 1 KiB aligned
  const uint32_t raw = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar = raw + kRawBytes;
  float* xbuf = reinterpret_cast<float*>(smem_raw + (raw - smem_u32(smem_raw)) + kRawBytes + 1024);
  constexpr uint32_t cbits = (LOG2K % 2 == 0) ? (uint32_t)(127 - LOG2K / 2) << 23
                                              : 0x3FB504F3u - ((uint32_t)((LOG2K + 1) / 2) << 23);
  const int t = threadIdx.x % T;              // thread within the row
  const int rs = threadIdx.x / T;             // row slot
  const int lo5 = t & 31, hi = t >> 5;
  float* bufA = xbuf + (size_t)rs * K;
  float* bufB = xbuf + (size_t)(ROWS + rs) * K;
  const int64_t row_iters = (p.M + ROWS - 1) / ROWS;

  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  __syncthreads();
  griddep_wait();
  griddep_launch_dependents();
  // this thread's 64 bytes inside the box: segment (t >> 1) of row slot rs, 16-byte pieces 4 (t & 1) + i,
  // stored at piece index ^ (segment & 7)
  const uint32_t seg = (uint32_t)rs * (K / 64) + (uint32_t)(t >> 1);
  const uint32_t raw_mine = raw + seg * 128u;
  const uint32_t raw_swz = seg & 7u;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmx);
    if ((int64_t)blockIdx.x < row_iters) {
      mbar_arrive_expect_tx(bar, kRawBytes);
      tma_load_3d(raw, &tmx, 0, 0, (int)((int64_t)blockIdx.x * ROWS), bar);
    }
  }

  uint4 sg[4] = {};
  if (SIGNS) {
    const uint4* sp = reinterpret_cast<const uint4*>(p.signs + (int64_t)t * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) sg[j] = __ldg(sp + j);
  }
  // shared-memory addresses that do not change from row to row
  const uint32_t a_w = smem_u32(bufA) + (uint32_t)t * 128u;                     // transpose 1, writes
  uint32_t a_r[8];                                                               // transpose 1, reads: row j + 32 hi
#pragma unroll
  for (int m = 0; m < 8; ++m)
    a_r[m] = smem_u32(bufA) + (uint32_t)hi * 4096u + (uint32_t)(((lo5 >> 2) ^ m) << 4) + (uint32_t)((lo5 & 3) << 2);
  uint32_t b_w[4];                                                               // transpose 2, writes
#pragma unroll
  for (int m = 0; m < 4; ++m)
    b_w[m] = smem_u32(bufB) + (uint32_t)hi * 4096u + (uint32_t)(((lo5 >> 2) ^ m) << 4) + (uint32_t)((lo5 & 3) << 2);
  const uint32_t b_r = smem_u32(bufB);                                           // transpose 2, reads

  uint32_t parity = 0;
  for (int64_t it = blockIdx.x; it < row_iters; it += gridDim.x) {
    const int64_t row = it * ROWS + rs;
    const bool live = row < p.M;                      // (rows beyond M arrive as zeros)
    const bool ok = mbar_wait(bar, parity, SITE_RQ_FULL);
    parity ^= 1u;
    uint64_t P[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 q = lds128(raw_mine + ((((uint32_t)(t & 1) * 4u + (uint32_t)j) ^ raw_swz) << 4));
      rq::unpack_stage1(SIGNS ? rq::apply_signs(q, sg[j]) : q, P + 4 * j);
    }
    rq::fwht32_stages_2_to_16(P);                                   // strides 1..16
    // ---- transpose 1
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      float a0, a1, a2, a3;
      rq::unpack2(P[2 * c], a0, a1);
      rq::unpack2(P[2 * c + 1], a2, a3);
      asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a_w + (uint32_t)((c ^ (t & 7)) << 4)), "f"(a0), "f"(a1),
                   "f"(a2), "f"(a3)
                   : "memory");
    }
    // (also: every thread has taken its bytes of the bf16 box; a lost load ends the loop for all)
    if (!__syncthreads_and(ok)) break;
    if (threadIdx.x == 0 && it + gridDim.x < row_iters) {
      mbar_arrive_expect_tx(bar, kRawBytes);
      tma_load_3d(raw, &tmx, 0, 0, (int)((it + gridDim.x) * ROWS), bar);
    }
    {
      float v[32];
#pragma unroll
      for (int j = 0; j < 32; ++j)
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[j]) : "r"(a_r[j & 7] + (uint32_t)(j * 128)) : "memory");
      // strides 32..256 on pairs (v[k], v[k + 16]); stride 512 inside the pairs
#pragma unroll
      for (int k = 0; k < 16; ++k) P[k] = rq::pack2(v[k], v[k + 16]);
      rq::fwht32_stages_2_to_16(P);
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        float lo, hi2;
        rq::unpack2(P[k], lo, hi2);
        v[k] = __fadd_rn(lo, hi2);
        v[k + 16] = __fsub_rn(lo, hi2);
      }
      // ---- transpose 2: value j is element lo5 + 32 j + 1024 hi of the row
#pragma unroll
      for (int j = 0; j < 32; ++j)
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(b_w[j & 3] + (uint32_t)(j * 128)), "f"(v[j]) : "memory");
    }
    __syncthreads();
    // ---- phase 3: runs of RUN consecutive values at RUN * t + 1024 * j2
    uint64_t E[NJ][RUN / 2];
#pragma unroll
    for (int j2 = 0; j2 < NJ; ++j2) {
#pragma unroll
      for (int h = 0; h < RUN / 4; ++h) {
        const uint32_t ci = (uint32_t)(j2 * 256 + t * (RUN / 4) + h);              // 16-byte piece of the row
        float a0, a1, a2, a3;
        asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(a0), "=f"(a1), "=f"(a2), "=f"(a3)
                     : "r"(b_r + ((ci ^ ((ci >> 3) & 3u)) << 4))
                     : "memory");
        E[j2][2 * h] = rq::pack2(a0, a1);
        E[j2][2 * h + 1] = rq::pack2(a2, a3);
      }
    }
#pragma unroll
    for (int hb = 1; hb < NJ; hb <<= 1) {                          // strides 1024 (and 2048)
#pragma unroll
      for (int j2 = 0; j2 < NJ; ++j2) {
        if ((j2 & hb) == 0) {
#pragma unroll
          for (int i = 0; i < RUN / 2; ++i) {
            const uint64_t a = E[j2][i], b = E[j2 + hb][i];
            E[j2][i] = rq::add2(a, b);
            E[j2 + hb][i] = rq::sub2(a, b);
          }
        }
      }
    }
    // ---- quantise: run j2 belongs to group (t >> HB) + 32 j2; the NJ lanes t, t^1 (, t^2, t^3) share it
#pragma unroll
    for (int j2 = 0; j2 < NJ; ++j2) {
      float m = 0.f;
#pragma unroll
      for (int i = 0; i < RUN / 2; ++i) {
        float lo, hi2;
        rq::unpack2(E[j2][i], lo, hi2);
        asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m) : "f"(lo), "f"(hi2));
      }
#pragma unroll
      for (int d = 1; d < NJ; d <<= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
      const float c = __uint_as_float(cbits);
      const uint32_t ef = __float_as_uint(__fmul_rn(m, c)) >> 23;
      const uint32_t sc = ef > 2u ? ef - 2u : 0u;
      float r[RUN];
      if (ef >= 27u && ef <= 250u) {
        const float c2 = __uint_as_float(cbits + ((127u - sc) << 23));
        const uint64_t cc = rq::pack2(c2, c2);
#pragma unroll
        for (int i = 0; i < RUN / 2; ++i) rq::unpack2(rq::mul2(E[j2][i], cc), r[2 * i], r[2 * i + 1]);
      } else {
        const float p2 = __uint_as_float((254u - sc) << 23);
        const uint64_t cc = rq::pack2(c, c), pp = rq::pack2(p2, p2);
#pragma unroll
        for (int i = 0; i < RUN / 2; ++i) rq::unpack2(rq::mul2(rq::mul2(E[j2][i], cc), pp), r[2 * i], r[2 * i + 1]);
      }
      uint32_t w[RUN / 8];
#pragma unroll
      for (int i = 0; i < RUN / 8; ++i)
        w[i] = rq::pack_e2m1x8(r[8 * i], r[8 * i + 1], r[8 * i + 2], r[8 * i + 3], r[8 * i + 4], r[8 * i + 5], r[8 * i + 6],
                               r[8 * i + 7]);
      if (live) {
        const int g = (t >> HB) + 32 * j2;
        uint8_t* dst = p.codes + row * (K >> 1) + g * 16 + (t & (NJ - 1)) * (RUN / 2);
        if (RUN == 8) *reinterpret_cast<uint32_t*>(dst) = w[0];
        else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[RUN / 8 - 1]);
        if ((t & (NJ - 1)) == 0) {
          if (p.layout == BRO_LAYOUT_GEMM) {
            const int64_t off = ((row >> 7) * p.scale_kblocks + (g >> 2)) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4 + (g & 3);
            p.scales[off] = (uint8_t)sc;
          } else {
            p.scales[row * (K >> 5) + g] = (uint8_t)sc;
          }
        }
      }
    }
  }
}

// 3-D view of x for the kernel above: {64 bf16 (128 bytes), K / 64 segments, M rows}, box = whole rows.
bro_status make_row_map(CUtensorMap* map, const void* x, int64_t M, int64_t K, int64_t ldx, int box_rows);

inline bro_status launch(const void* x, int64_t M, int64_t K, int64_t ldx, const void* signs, void* codes,
                         void* scales, float* mse, int format, bro_layout layout, int64_t scale_kblocks, int sm_count, cudaStream_t st,
                         float* deq = nullptr, int64_t ldd = 0, uint32_t* rowstats = nullptr, bool range_pass = false) {
  Params p;
  p.deq = deq;
  p.ldd = ldd;
  p.rowstats = rowstats;
  p.range_pass = range_pass ? 1 : 0;
  p.x = static_cast<const uint16_t*>(x);
  p.M = M;
  p.K = K;
  p.ldx = ldx;
  p.codes = static_cast<uint8_t*>(codes);
  p.scales = static_cast<uint8_t*>(scales);
  p.scale_kblocks = scale_kblocks;
  p.layout = (int)layout;
  p.signs = static_cast<const uint16_t*>(signs);
  p.mse = mse;
  p.format = format;
  int lg = 0;
  while (((int64_t)1 << lg) < K) ++lg;
  p.log2k = lg;
  p.threads_per_row = (int)(K / 32);
  int threads = p.threads_per_row < 256 ? 256 : p.threads_per_row;
  p.rows_per_iter = threads / p.threads_per_row;
  const size_t smem = K > 1024 ? (size_t)p.rows_per_iter * K * sizeof(float) : 0;
  if (layout == BRO_LAYOUT_GEMM && !mse && !deq && !range_pass && format != rq::kFormatScaleOnly) {
    // padding rows / groups of the tiled scale buffer must read as 0
    const size_t bytes = (size_t)((M + 127) / 128) * (size_t)scale_kblocks * 512;
    if (cudaMemsetAsync(scales, 0, bytes, st) != cudaSuccess) return BRO_ERR_CUDA;
  }
  if ((K == 2048 || K == 4096) && !mse && !deq && !range_pass && format != rq::kFormatScaleOnly) {
    // codes path at these sizes: all stages in registers, two shared-memory transposes
    const int rows = (int)(128 / (K / 32));
    const int64_t iters2 = (M + rows - 1) / rows;
    const size_t smem2 = (size_t)2 * rows * K * sizeof(float) + (size_t)rows * K * 2 + 2048;   // fp32 buffers, bf16 box, barrier, alignment
    CUtensorMap tmx;
    const bro_status mrc = make_row_map(&tmx, x, M, K, ldx, rows);
    if (mrc != BRO_OK) return mrc;
    auto go2 = [&](auto kernel) -> bro_status {
      static DeviceOnce once;                                             // (one per instantiation)
      int per_sm = 1;
      const bro_status rc = device_once(once, &per_sm, [&](int* n) {
        if (!cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2),
                     "cudaFuncSetAttribute(rotate_quantize_global_smem)"))
          return BRO_ERR_CUDA;
        return cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, kernel, 128, smem2),
                       "occupancy(rotate_quantize_global_smem)")
                   ? BRO_OK
                   : BRO_ERR_CUDA;
      });
      if (rc != BRO_OK) return rc;
      const int64_t cap = (int64_t)sm_count * per_sm;
      const unsigned grid2 = (unsigned)(iters2 < cap ? iters2 : cap);
      return cuda_ok(launch_kernel(kernel, grid2, 128u, smem2, st, 1, tmx, p), "rotate_quantize_global_smem launch") ? BRO_OK
                                                                                                                 : BRO_ERR_CUDA;
    };
    if (K == 4096) return signs ? go2(rotate_quantize_global_smem_kernel<12, true>) : go2(rotate_quantize_global_smem_kernel<12, false>);
    return signs ? go2(rotate_quantize_global_smem_kernel<11, true>) : go2(rotate_quantize_global_smem_kernel<11, false>);
  }
  const int64_t iters = (M + p.rows_per_iter - 1) / p.rows_per_iter;
  const int64_t max_grid = (int64_t)sm_count * (threads <= 512 ? 2 : 1);
  const int grid = (int)(iters < max_grid ? iters : max_grid);
  auto go = [&](auto kernel) -> bro_status {
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return BRO_ERR_CUDA;
    return cuda_ok(launch_kernel(kernel, (unsigned)grid, (unsigned)threads, smem, st, 1, p),
                   "rotate_quantize_global launch")
               ? BRO_OK
               : BRO_ERR_CUDA;
  };
  if (threads <= 256) return go(rotate_quantize_global_kernel<256>);
  if (threads <= 512) return go(rotate_quantize_global_kernel<512>);
  return go(rotate_quantize_global_kernel<1024>);
}

}  // namespace rqg
}  // namespace bro
