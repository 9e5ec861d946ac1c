// Kernel 1 (register-streaming form): fused block-Hadamard rotation + MXFP4 quantisation
// (paper Sec. 4.3 Eq. 1, Sec. 4.1) without a shared-memory stage.
//
// Same arithmetic contract as rotate_quantize.cuh (whose helpers it reuses): a thread owns one MX
// group of 32 consecutive channels, butterflies with ascending stride in fp32, one multiply by
// fp32(1/sqrt(block)), amax -> E8M0 exponent, round-to-nearest-even E2M1 codes.
//
// What differs is how the bytes travel.  The 32 lanes of a warp take 32 consecutive groups of one
// row (2 KiB of contiguous bf16), each lane loading its 64 bytes with four 16-byte loads straight
// into registers, and the loads of the warp's NEXT task are issued before the current one is
// computed.  Nothing goes through shared memory: in the TMA-ring form the shared-memory port carries
// every byte twice (TMA write, then the consumers' loads) and all consumer warps wake on the same
// barrier, which together cost about a third of its run time on a [16384, 4096] tensor; here more
// warps are resident and they drift apart, so loads, arithmetic and stores of different warps
// overlap.  Blocks of 64 / 128 channels pair lanes l ^ 1 (and l ^ 2) for their last one / two stages,
// each lane exchanging half of its values (rq::cross_lane_split); the per-group error kernels keep the
// whole group in one lane (rq::cross_lane_stage).  Blocks of 2..16 channels (a rotation inside the MX
// group, LOG2B = 1..4) stop the butterfly early (rq::fwht32_stages_below).
#pragma once

#include "bro_common.cuh"
#include "rotate_quantize.cuh"

namespace bro {
namespace rqd {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct Params {
  const uint16_t* x;
  int64_t M, K, ldx;
  uint8_t* codes;               // [M, K/2]
  uint8_t* scales;
  int64_t scale_kblocks;        // tensor-core layout: 512-byte blocks per 128-row block
  int layout;                   // bro_layout
  const uint16_t* signs;        // [K] bf16 +-1 (kernels with SIGNS) or nullptr
  int rows_padded;              // rows the task grid covers (a multiple of 128 for the tensor-core layout)
  int groups_padded;            // groups per row it covers (scale padding included)
  int chunks_per_row;           // ceil(groups_padded / 32)
  int total_tasks;              // rows_padded * chunks_per_row; one task = one warp, 32 groups of a row
  const uint16_t* up;           // PRODUCER kernels: the second operand of h = silu(x) * up, [M, K] with row stride ldu
  int64_t ldu;
  float* mse;                   // STATS kernels: [M, K/32] per-group quantisation error instead of codes/scales
  int format;                   // STATS kernels: which 4-bit format (see rq::group_error), or
                                // rq::kFormatScaleOnly: write the E8M0 byte to scales[M, K/32] and nothing else
};

// ---- the producer fused in front of the rotation (PRODUCER = 1) ------------------------------------------
// The online rotation sits before down_proj (paper Sec. 4.3, "Reduced online computing"), whose input in
// the LLaMA-family models is h = silu(gate) * up.  Computing h inside this kernel saves writing it to HBM
// and reading it back (4 of 8.5 bytes per element).  The arithmetic is a fixed sequence of IEEE fp32
// operations (one rounding each), so that it can be reproduced bit for bit elsewhere:
//   t = -|g|;  n = rint(t log2e);  r = fma(n, -ln2_hi, t);  r = fma(n, -ln2_lo, r);
//   p = 1 + r (1 + r (1/2 + r (1/6 + r (1/24 + r (1/120 + r/720)))))  (Horner, fma);  e = p 2^n  (0 if t < -86);
//   h = bf16_rne((g * ((g >= 0 ? 1 : e) / (1 + e))) * u).
__device__ __forceinline__ float silu_mul(float g, float u) {
  const float t = -fabsf(g);
  const float n = rintf(__fmul_rn(t, __uint_as_float(0x3FB8AA3Bu)));
  float r = __fmaf_rn(n, -__uint_as_float(0x3F317218u), t);
  r = __fmaf_rn(n, -__uint_as_float(0xB102E308u), r);
  float p = __uint_as_float(0x3AB60B61u);
  p = __fmaf_rn(p, r, __uint_as_float(0x3C088889u));
  p = __fmaf_rn(p, r, __uint_as_float(0x3D2AAAABu));
  p = __fmaf_rn(p, r, __uint_as_float(0x3E2AAAABu));
  p = __fmaf_rn(p, r, 0.5f);
  p = __fmaf_rn(p, r, 1.0f);
  p = __fmaf_rn(p, r, 1.0f);
  float e = __uint_as_float(__float_as_uint(p) + ((uint32_t)(int)n << 23));   // p in [0.70, 1.42], n in [-124, 0]: exact
  e = t >= -86.0f ? e : 0.0f;
  const float s = __fdiv_rn(g >= 0.0f ? 1.0f : e, __fadd_rn(1.0f, e));
  return __fmul_rn(__fmul_rn(g, s), u);
}
// 8 bf16 gates and 8 bf16 ups -> 8 bf16 values of h
__device__ __forceinline__ uint4 swiglu_bf16x8(uint4 g, uint4 u) {
  const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
  uint32_t h[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float lo = silu_mul(__uint_as_float(gw[k] << 16), __uint_as_float(uw[k] << 16));
    const float hi = silu_mul(__uint_as_float(gw[k] & 0xFFFF0000u), __uint_as_float(uw[k] & 0xFFFF0000u));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(h[k]) : "f"(hi), "f"(lo));
  }
  return make_uint4(h[0], h[1], h[2], h[3]);
}

// STATS: nothing is quantised to memory; the kernel writes the per-group quantisation error
// (rq::group_error) — the analysis behind the paper's regular-block / outlier-block comparison.
// PRODUCER: the rotated tensor is h = silu(x) * up (see silu_mul), computed here from the two bf16 inputs.
template <int LOG2B, bool SIGNS, bool STATS, bool PRODUCER = false>
__global__ void __launch_bounds__(kThreads, PRODUCER ? 2 : 3)
rotate_quantize_direct_kernel(const Params p) {
  const int lane = threadIdx.x & 31;
  const int num_warps = (int)gridDim.x * kWarps;
  const int ng = (int)(p.K >> 5);
  constexpr uint32_t cbits = rq::norm_bits<LOG2B>();

  griddep_wait();               // x may be written, codes/scales still read, by the kernel before
  // (only now: a dependent that starts early may then rely on everything older than this kernel)
  griddep_launch_dependents();

  // task -> (row, chunk); advanced incrementally (no division in the loop)
  int task = (int)blockIdx.x * kWarps + (int)(threadIdx.x >> 5);
  int row = task / p.chunks_per_row, chunk = task - row * p.chunks_per_row;
  const int step_row = num_warps / p.chunks_per_row, step_chunk = num_warps - step_row * p.chunks_per_row;

  // blocks of 64 / 128 (codes path): odd lanes hold their group with the 32-byte halves exchanged
  constexpr bool kSplit = LOG2B >= 6 && !STATS;
  const int hswz = (kSplit && (lane & 1)) ? 2 : 0;

  auto load = [&](int r, int c, uint4 (&q)[4], uint4 (&qu)[4]) {
    const int g = c * 32 + lane;
    if (r < p.M && g < ng) {
      const uint4* src = reinterpret_cast<const uint4*>(p.x + (int64_t)r * p.ldx + (int64_t)g * 32);
#pragma unroll
      for (int j = 0; j < 4; ++j) q[j] = __ldg(src + (j ^ hswz));
      if (PRODUCER) {
        const uint4* usrc = reinterpret_cast<const uint4*>(p.up + (int64_t)r * p.ldu + (int64_t)g * 32);
#pragma unroll
        for (int j = 0; j < 4; ++j) qu[j] = __ldg(usrc + (j ^ hswz));
      }
      if (SIGNS && !PRODUCER) {
        const uint4* sp = reinterpret_cast<const uint4*>(p.signs + (int64_t)g * 32);
#pragma unroll
        for (int j = 0; j < 4; ++j) q[j] = rq::apply_signs(q[j], __ldg(sp + (j ^ hswz)));
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) q[j] = make_uint4(0u, 0u, 0u, 0u);   // padding quantises to zeros
      if (PRODUCER) {
#pragma unroll
        for (int j = 0; j < 4; ++j) qu[j] = make_uint4(0u, 0u, 0u, 0u);   // (silu(0) * 0 = 0)
      }
    }
  };

  uint4 cur[4], nxt[4], cur_u[4], nxt_u[4];
  if (task < p.total_tasks) load(row, chunk, cur, cur_u);
  while (task < p.total_tasks) {
    // the next task of this warp: issue its loads now, use them in the next iteration
    const int ntask = task + num_warps;
    int nrow = row + step_row, nchunk = chunk + step_chunk;
    if (nchunk >= p.chunks_per_row) { nchunk -= p.chunks_per_row; ++nrow; }
    if (ntask < p.total_tasks) load(nrow, nchunk, nxt, nxt_u);

    if (PRODUCER) {
      // h = silu(gate) * up, rounded to bf16: from here on the kernel is the plain one on h
#pragma unroll
      for (int j = 0; j < 4; ++j) cur[j] = swiglu_bf16x8(cur[j], cur_u[j]);
      if (SIGNS && row < p.M && chunk * 32 + lane < ng) {
        const uint4* sp = reinterpret_cast<const uint4*>(p.signs + (int64_t)(chunk * 32 + lane) * 32);
#pragma unroll
        for (int j = 0; j < 4; ++j) cur[j] = rq::apply_signs(cur[j], __ldg(sp + (j ^ hswz)));
      }
    }

    uint64_t P[16];
#pragma unroll
    for (int j = 0; j < 4; ++j) rq::unpack_stage1(cur[j], P + 4 * j);
    const int g = chunk * 32 + lane;
    const bool live = row < p.M && g < ng;
    if constexpr (kSplit) {
      rq::fwht32_stages_2_to_8(P);
      uint32_t wx[2], wy[2], sx, sy;
      rq::cross_lane_split<LOG2B>(P, lane, cbits, wx, sx, wy, sy);
      // the lanes of a block share `live` (K is a multiple of the block); this lane's 16 codes of
      // group X and of group Y are 8 bytes each, at byte (lane & 1) * 8 of the group's 16
      const int gb = chunk * 32 + (LOG2B == 6 ? (lane & ~1) : (lane & ~3));
      const int gx = gb + (LOG2B == 6 ? 0 : ((lane >> 1) & 1));
      const int gy = gx + (LOG2B == 6 ? 1 : 2);
      if (live) {
        uint8_t* rowp = p.codes + (int64_t)row * (p.K >> 1) + (lane & 1) * 8;
        *reinterpret_cast<uint2*>(rowp + (int64_t)gx * 16) = make_uint2(wx[0], wx[1]);
        *reinterpret_cast<uint2*>(rowp + (int64_t)gy * 16) = make_uint2(wy[0], wy[1]);
      }
      // scale bytes of groups 4j..4j+3 -> one 32-bit word in the lane with lane % 4 == 0
      uint32_t sb;
      if (LOG2B == 6) {
        const uint32_t mine = live ? (sx | (sy << 8)) : 0u;          // groups (2i, 2i+1) of this lane pair
        sb = mine | (__shfl_xor_sync(0xFFFFFFFFu, mine, 2) << 16);
      } else {
        const uint32_t mine = live ? (sx | (sy << 16)) : 0u;         // groups (0, 2) or (1, 3) of the block
        sb = mine | (__shfl_xor_sync(0xFFFFFFFFu, mine, 2) << 8);
      }
      if ((lane & 3) == 0 && g < p.groups_padded) {
        if (p.layout == BRO_LAYOUT_GEMM) {
          const int64_t off = ((int64_t)(row >> 7) * p.scale_kblocks + (g >> 2)) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4;
          *reinterpret_cast<uint32_t*>(p.scales + off) = sb;
        } else if (row < p.M && g < ng) {
          // (ng is a multiple of 2 or 4 here, so the 4 groups of this word exist whenever g + 4 <= ng)
          uint8_t* dst = p.scales + (int64_t)row * ng + g;
          if (g + 4 <= ng && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
            *reinterpret_cast<uint32_t*>(dst) = sb;
          } else {
            for (int i = 0; i < 4 && g + i < ng; ++i) dst[i] = (uint8_t)(sb >> (8 * i));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) { cur[j] = nxt[j]; if (PRODUCER) cur_u[j] = nxt_u[j]; }
      task = ntask;
      row = nrow;
      chunk = nchunk;
      continue;
    }
    if constexpr (LOG2B >= 5) rq::fwht32_stages_2_to_16(P);
    else rq::fwht32_stages_below<LOG2B>(P);          // a rotation inside the MX group stops early
    if (LOG2B >= 6) rq::cross_lane_stage(P, 1, (lane & 1) != 0);
    if (LOG2B >= 7) rq::cross_lane_stage(P, 2, (lane & 2) != 0);
    if (STATS) {
      if (p.format == rq::kFormatScaleOnly) {
        const uint32_t sbyte = rq::group_scale_byte(P, cbits);
        if (live) p.scales[(int64_t)row * ng + g] = (uint8_t)sbyte;
      } else {
        const float e = rq::group_error(P, cbits, p.format);
        if (live) p.mse[(int64_t)row * ng + g] = e;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) { cur[j] = nxt[j]; if (PRODUCER) cur_u[j] = nxt_u[j]; }
      task = ntask;
      row = nrow;
      chunk = nchunk;
      continue;
    }
    uint32_t w[4];
    const uint32_t s = rq::quantize_group(P, cbits, w);
    if (live)
      *reinterpret_cast<uint4*>(p.codes + (int64_t)row * (p.K >> 1) + (int64_t)g * 16) = make_uint4(w[0], w[1], w[2], w[3]);
    // scale bytes of 4 consecutive groups -> one 32-bit word in the lane with g % 4 == 0
    uint32_t sb = live ? s : 0u;
    sb |= __shfl_xor_sync(0xFFFFFFFFu, sb, 1) << 8;
    sb |= __shfl_xor_sync(0xFFFFFFFFu, sb, 2) << 16;
    if ((lane & 3) == 0 && g < p.groups_padded) {
      if (p.layout == BRO_LAYOUT_GEMM) {
        // 512-byte block (row / 128, g / 4): byte (r % 32) * 16 + ((r % 128) / 32) * 4 + g % 4
        const int64_t off = ((int64_t)(row >> 7) * p.scale_kblocks + (g >> 2)) * 512 + (row & 31) * 16 + ((row & 127) >> 5) * 4;
        *reinterpret_cast<uint32_t*>(p.scales + off) = sb;
      } else if (row < p.M) {
        uint8_t* dst = p.scales + (int64_t)row * ng + g;
        if (g + 4 <= ng && (reinterpret_cast<uintptr_t>(dst) & 3) == 0) {
          *reinterpret_cast<uint32_t*>(dst) = sb;
        } else {
          for (int i = 0; i < 4 && g + i < ng; ++i) dst[i] = (uint8_t)(sb >> (8 * i));
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) { cur[j] = nxt[j]; if (PRODUCER) cur_u[j] = nxt_u[j]; }
    task = ntask;
    row = nrow;
    chunk = nchunk;
  }
}

// Rows x padded groups must fit 31 bits of task index; larger problems use the TMA-ring kernel.
inline bool supports(int64_t M, int64_t K, bro_layout layout, int64_t scale_kblocks) {
  const int64_t rows = layout == BRO_LAYOUT_GEMM ? (M + 127) / 128 * 128 : M;
  const int64_t groups = layout == BRO_LAYOUT_GEMM ? scale_kblocks * 4 : K / 32;
  return rows * ((groups + 31) / 32) < ((int64_t)1 << 30);
}

template <int LOG2B, bool SIGNS, bool STATS, bool PRODUCER = false>
inline bro_status launch_one(Params& p, int sm_count, cudaStream_t st) {
  auto kernel = rotate_quantize_direct_kernel<LOG2B, SIGNS, STATS, PRODUCER>;
  static DeviceOnce once;            // (one per template instantiation)
  int blocks_per_sm = 1;
  const bro_status rc = device_once(once, &blocks_per_sm, [&](int* n) {
    return cuda_ok(cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, kernel, kThreads, 0), "occupancy(rotate_quantize_direct)")
               ? BRO_OK
               : BRO_ERR_CUDA;
  });
  if (rc != BRO_OK) return rc;
  const int64_t want = ((int64_t)p.total_tasks + kWarps - 1) / kWarps;
  const int64_t cap = (int64_t)sm_count * blocks_per_sm;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  return cuda_ok(launch_kernel(kernel, grid, kThreads, 0, st, 1, p), "rotate_quantize_direct launch") ? BRO_OK
                                                                                                       : BRO_ERR_CUDA;
}

template <bool STATS, bool PRODUCER = false>
inline bro_status launch_any(Params& p, int log2b, int sm_count, cudaStream_t st) {
  if constexpr (!STATS) {       // rotations inside the MX group (blocks of 2..16): the quantising kernels only
    if (p.signs) {
      switch (log2b) {
        case 1: return launch_one<1, true, false, PRODUCER>(p, sm_count, st);
        case 2: return launch_one<2, true, false, PRODUCER>(p, sm_count, st);
        case 3: return launch_one<3, true, false, PRODUCER>(p, sm_count, st);
        case 4: return launch_one<4, true, false, PRODUCER>(p, sm_count, st);
        default: break;
      }
    } else {
      switch (log2b) {
        case 1: return launch_one<1, false, false, PRODUCER>(p, sm_count, st);
        case 2: return launch_one<2, false, false, PRODUCER>(p, sm_count, st);
        case 3: return launch_one<3, false, false, PRODUCER>(p, sm_count, st);
        case 4: return launch_one<4, false, false, PRODUCER>(p, sm_count, st);
        default: break;
      }
    }
  }
  if (p.signs) {
    switch (log2b) {
      case 5: return launch_one<5, true, STATS, PRODUCER>(p, sm_count, st);
      case 6: return launch_one<6, true, STATS, PRODUCER>(p, sm_count, st);
      default: return launch_one<7, true, STATS, PRODUCER>(p, sm_count, st);
    }
  }
  switch (log2b) {
    case 5: return launch_one<5, false, STATS, PRODUCER>(p, sm_count, st);
    case 6: return launch_one<6, false, STATS, PRODUCER>(p, sm_count, st);
    default: return launch_one<7, false, STATS, PRODUCER>(p, sm_count, st);
  }
}

// `up` != nullptr: x is the gate and the rotated tensor is silu(x) * up (the fused producer).
inline bro_status launch(const void* x, int64_t M, int64_t K, int64_t ldx, int log2b, const void* signs, void* codes,
                         void* scales, bro_layout layout, int64_t scale_kblocks, int sm_count, cudaStream_t st,
                         const void* up = nullptr, int64_t ldu = 0) {
  Params p;
  p.x = static_cast<const uint16_t*>(x);
  p.up = static_cast<const uint16_t*>(up);
  p.ldu = ldu;
  p.M = M; p.K = K; p.ldx = ldx;
  p.codes = static_cast<uint8_t*>(codes);
  p.scales = static_cast<uint8_t*>(scales);
  p.scale_kblocks = scale_kblocks;
  p.layout = (int)layout;
  p.signs = static_cast<const uint16_t*>(signs);
  p.mse = nullptr;
  p.format = 0;
  p.rows_padded = (int)(layout == BRO_LAYOUT_GEMM ? (M + 127) / 128 * 128 : M);
  p.groups_padded = (int)(layout == BRO_LAYOUT_GEMM ? scale_kblocks * 4 : K / 32);
  p.chunks_per_row = (p.groups_padded + 31) / 32;
  p.total_tasks = p.rows_padded * p.chunks_per_row;
  return up ? launch_any<false, true>(p, log2b, sm_count, st) : launch_any<false>(p, log2b, sm_count, st);
}

// Per-group quantisation error only: mse[M, K/32] (fp32) — or, with format = rq::kFormatScaleOnly, the
// per-group scale byte only: scale_bytes[M, K/32].
inline bro_status launch_stats(const void* x, int64_t M, int64_t K, int64_t ldx, int log2b, const void* signs,
                               int format, float* mse, uint8_t* scale_bytes, int sm_count, cudaStream_t st) {
  Params p;
  p.x = static_cast<const uint16_t*>(x);
  p.up = nullptr;
  p.ldu = 0;
  p.M = M; p.K = K; p.ldx = ldx;
  p.codes = nullptr;
  p.scales = scale_bytes;
  p.scale_kblocks = 0;
  p.layout = (int)BRO_LAYOUT_CANONICAL;
  p.signs = static_cast<const uint16_t*>(signs);
  p.mse = mse;
  p.format = format;
  p.rows_padded = (int)M;
  p.groups_padded = (int)(K / 32);
  p.chunks_per_row = (p.groups_padded + 31) / 32;
  p.total_tasks = p.rows_padded * p.chunks_per_row;
  return launch_any<true>(p, log2b, sm_count, st);
}

}  // namespace rqd
}  // namespace bro
