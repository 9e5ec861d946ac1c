// Simulated ("fake") quantisation: rotate, quantise to one of the compared 4-bit formats, dequantise.
// The paper evaluates every method this way (Sec. 3.1, experimental setup: MX quantisation is
// simulated, no native FP4 GEMM is run), and its format study (Sec. 3.2 / Fig. 2, Sec. 4.1 / Fig. 3)
// compares MXFP4 with BFP4, MXINT4 and BINT4 on the same tensors.  This kernel gives those tensors at
// full bandwidth: out[m, k] = deq(Q_format((x R)[m, :]))_k as fp32, in the rotated domain.
//
// One thread owns one MX group of 32 channels (64 bytes of bf16), a warp 32 consecutive groups of a
// row; the rotation is the same fixed-order fp32 butterfly as in the quantising kernels (stages of
// stride 1..16 in registers, stride 32 / 64 through one / two shuffles for blocks of 64 / 128), or
// none at all (LOG2B = 0: the identity, "before rotation"), or a rotation inside the MX group
// (LOG2B = 1..4: blocks of 2..16 channels — the paper's Sec. 5.2 sweeps the rotation dimension below as
// well as above the MX group), which simply stops the butterfly early.  Every dequantised value is exactly
// representable in fp32 (a 3-bit element times a power of two or an 11-bit fp16 scale), so the result
// can be compared bit for bit with an evaluation in higher precision.
//
// An analysis path: 2 bytes read and 4 written per element.  A thread's 128 output bytes go through a
// per-warp shared-memory buffer (16-byte pieces XOR-swizzled with the lane, conflict-free both ways) so
// that every store instruction of the warp writes 512 contiguous bytes of the row.
#pragma once

#include "bro_common.cuh"
#include "rotate_quantize.cuh"

namespace bro {
namespace fq {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// The 32 values of one group (P holds the un-normalised butterfly output, y = P * c) dequantised
// under `format`: 0 MXFP4 (E2M1, scale 2^E, E = floor(log2 amax) - 2), 1 BFP4 (E2M1, scale
// fp16(amax / 6)), 2 MXINT4 (k / 4, |k| <= 7, scale 2^E, E = floor(log2 amax)), 3 BINT4 (|k| <= 7,
// scale fp16(amax / 7)).  Decisions are taken exactly as in rq::group_error: magnitudes scaled by an
// exact power of two, or divided by the fp16 scale in fp32, then rounded to nearest even, saturating.
__device__ __forceinline__ void group_dequant(const uint64_t (&P)[16], uint32_t cbits, int format, float (&out)[32]) {
  const float c = __uint_as_float(cbits);
  const uint64_t cc = rq::pack2(c, c);
  float y[32];
#pragma unroll
  for (int k = 0; k < 16; ++k) rq::unpack2(rq::mul2(P[k], cc), y[2 * k], y[2 * k + 1]);
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) m = fmaxf(m, fabsf(y[i]));
  const uint32_t ef = __float_as_uint(m) >> 23;
  auto e2m1 = [](float r0, float r1, float& q0, float& q1) {
    uint32_t h;
    asm("{ .reg .b8 b; cvt.rn.satfinite.e2m1x2.f32 b, %2, %1; cvt.rn.f16x2.e2m1x2 %0, b; }" : "=r"(h) : "f"(r0), "f"(r1));
    q0 = __half2float(__ushort_as_half((unsigned short)(h & 0xFFFFu)));
    q1 = __half2float(__ushort_as_half((unsigned short)(h >> 16)));
  };
  if (format == 0 || format == 2) {
    const uint32_t s = format == 0 ? (ef > 2u ? ef - 2u : 0u) : ef;
    // 2^-E and 2^E with E = s - 127 (2^-127 is a subnormal)
    const float inv = __uint_as_float(s <= 253u ? ((254u - s) << 23) : 0x00400000u);
    const float pe = __uint_as_float(s >= 1u ? (s << 23) : 0x00400000u);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
      const float r0 = __fmul_rn(fabsf(y[i]), inv), r1 = __fmul_rn(fabsf(y[i + 1]), inv);
      float q0, q1;
      if (format == 0) {
        e2m1(r0, r1, q0, q1);
      } else {
        q0 = 0.25f * (float)min(__float2int_rn(__fmul_rn(r0, 4.f)), 7);
        q1 = 0.25f * (float)min(__float2int_rn(__fmul_rn(r1, 4.f)), 7);
      }
      out[i] = copysignf(__fmul_rn(q0, pe), y[i]);
      out[i + 1] = copysignf(__fmul_rn(q1, pe), y[i + 1]);
    }
    return;
  }
  // fp16 scale: the fp32 quotient amax / qmax rounded to nearest-even fp16, saturating
  float sc;
  {
    const float quot = __fdiv_rn(m, format == 1 ? 6.f : 7.f);
    unsigned short hb;
    asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(hb) : "f"(quot));
    sc = __half2float(__ushort_as_half(hb));
  }
#pragma unroll
  for (int i = 0; i < 32; i += 2) {
    if (sc == 0.f) {                 // (a scale that rounds to zero gives an all-zero group)
      out[i] = 0.f;
      out[i + 1] = 0.f;
      continue;
    }
    const float r0 = __fdiv_rn(fabsf(y[i]), sc), r1 = __fdiv_rn(fabsf(y[i + 1]), sc);
    float q0, q1;
    if (format == 1) {
      e2m1(r0, r1, q0, q1);
    } else {
      q0 = (float)min(__float2int_rn(r0), 7);
      q1 = (float)min(__float2int_rn(r1), 7);
    }
    out[i] = copysignf(__fmul_rn(q0, sc), y[i]);
    out[i + 1] = copysignf(__fmul_rn(q1, sc), y[i + 1]);
  }
}

__device__ __forceinline__ void store_group(float* dst, const float (&out)[32]) {
#pragma unroll
  for (int j = 0; j < 8; ++j)
    reinterpret_cast<float4*>(dst)[j] = make_float4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
}

// ---- INT4 with one scale per ROW (Sec. 3.2 / Fig. 2: per-channel symmetric weights, per-token asymmetric
// activations).  Two passes over the input: the first leaves the row's range in `rowstats`, the second
// quantises with it.  rowstats[2 * row] = bits of max(-min(row), 0), rowstats[2 * row + 1] = bits of
// max(max(row), 0): both are non-negative floats, which order like their bit patterns, so an integer
// atomicMax onto zero-initialised words is an exact, order-independent reduction.
constexpr int kFormatRowSym = 4, kFormatRowAsym = 5, kFormatNone = 6;

__device__ __forceinline__ void group_range(const uint64_t (&P)[16], uint32_t cbits, float& neglo, float& hi) {
  const float c = __uint_as_float(cbits);
  const uint64_t cc = rq::pack2(c, c);
  neglo = 0.f;
  hi = 0.f;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float a, b;
    rq::unpack2(rq::mul2(P[k], cc), a, b);
    hi = fmaxf(hi, fmaxf(a, b));
    neglo = fmaxf(neglo, fmaxf(-a, -b));
  }
}

// The 32 values of a group under the row's scale.  Symmetric: |k| <= 7, scale fp16(amax / 7).  Asymmetric:
// codes 0..15 over [lo, hi] (the range always contains zero): scale fp16((hi - lo) / 15), zero point
// z = rint(-lo / scale) (at most 15), q = clamp(rint(y / scale) + z, 0, 15), value (q - z) scale.  Quotients
// are IEEE fp32 divisions; every result is an integer of at most 5 bits times an fp16 number, exact in fp32.
__device__ __forceinline__ void row_dequant(const uint64_t (&P)[16], uint32_t cbits, bool asym, float neglo, float hi,
                                            float (&out)[32]) {
  const float c = __uint_as_float(cbits);
  const uint64_t cc = rq::pack2(c, c);
  float y[32];
#pragma unroll
  for (int k = 0; k < 16; ++k) rq::unpack2(rq::mul2(P[k], cc), y[2 * k], y[2 * k + 1]);
  const float quot = asym ? __fdiv_rn(__fadd_rn(hi, neglo), 15.f) : __fdiv_rn(fmaxf(hi, neglo), 7.f);
  unsigned short hb;
  asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(hb) : "f"(quot));
  const float sc = __half2float(__ushort_as_half(hb));
  if (sc == 0.f) {                  // (a scale that rounds to zero gives an all-zero row)
#pragma unroll
    for (int i = 0; i < 32; ++i) out[i] = 0.f;
    return;
  }
  if (!asym) {
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      const float q = (float)min(__float2int_rn(__fdiv_rn(fabsf(y[i]), sc)), 7);
      out[i] = copysignf(__fmul_rn(q, sc), y[i]);
    }
    return;
  }
  const int z = min(__float2int_rn(__fdiv_rn(neglo, sc)), 15);
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    int q = __float2int_rn(__fdiv_rn(y[i], sc));
    q = max(-16, min(q, 31)) + z;
    q = max(0, min(q, 15));
    out[i] = __fmul_rn((float)(q - z), sc);
  }
}

struct Params {
  const uint16_t* x;
  int64_t M, K, ldx;
  const uint16_t* signs;        // [K] bf16 +-1 (kernels with SIGNS) or nullptr
  uint32_t* rowstats;           // [M, 2] the row ranges (see group_range): written when deq == nullptr and
                                // neither statistic is asked for, read by the per-row formats
  float* deq;                   // [M, K] fp32, row stride ldd — or nullptr, and then one of:
  int64_t ldd;
  float* mse;                   //   [M, K/32] per-group quantisation error (rq::group_error)
  uint8_t* scale_bytes;         //   [M, K/32] E8M0 byte of each group (rq::group_scale_byte)
  int format;
  int chunks_per_row;           // ceil((K / 32) / 32): one task = one warp, 32 groups of a row
  int64_t total_tasks;          // M * chunks_per_row
};

// LOG2B = 0: no rotation; 1..4: blocks of 2..16 inside the group; 5, 6, 7: blocks of 32, 64, 128.
template <int LOG2B, bool SIGNS>
__global__ void __launch_bounds__(kThreads, 2) fake_quantize_kernel(const Params p) {
  __shared__ __align__(16) float sbuf[kWarps][32 * 32];      // 4 KiB per warp
  const int lane = threadIdx.x & 31;
  float* wbuf = sbuf[threadIdx.x >> 5];
  const int ng = (int)(p.K >> 5);
  constexpr uint32_t cbits = LOG2B == 0 ? 0x3F800000u : rq::norm_bits<(LOG2B == 0 ? 5 : LOG2B)>();
  const bool full = p.deq != nullptr;             // (uniform over the grid)
  griddep_wait();
  griddep_launch_dependents();
  const int64_t num_warps = (int64_t)gridDim.x * kWarps;
  for (int64_t task = (int64_t)blockIdx.x * kWarps + (threadIdx.x >> 5); task < p.total_tasks; task += num_warps) {
    const int64_t row = task / p.chunks_per_row;
    const int g = (int)(task - row * p.chunks_per_row) * 32 + lane;
    const bool live = g < ng;      // (K is a multiple of the block, so the lanes of a block share `live`)
    uint64_t P[16];
    const uint4* src = reinterpret_cast<const uint4*>(p.x + row * p.ldx + (int64_t)g * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint4 q = live ? __ldg(src + j) : make_uint4(0u, 0u, 0u, 0u);
      if (SIGNS && live) q = rq::apply_signs(q, __ldg(reinterpret_cast<const uint4*>(p.signs + (int64_t)g * 32) + j));
      if (LOG2B == 0) {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int k = 0; k < 4; ++k)
          P[4 * j + k] = rq::pack2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xFFFF0000u));
      } else {
        rq::unpack_stage1(q, P + 4 * j);
      }
    }
    if (LOG2B >= 5) rq::fwht32_stages_2_to_16(P);
    if (LOG2B >= 2 && LOG2B <= 4) rq::fwht32_stages_below<(LOG2B >= 2 && LOG2B <= 4) ? LOG2B : 2>(P);
    if (LOG2B >= 6) rq::cross_lane_stage(P, 1, (lane & 1) != 0);
    if (LOG2B >= 7) rq::cross_lane_stage(P, 2, (lane & 2) != 0);
    if (!full && !p.mse && !p.scale_bytes) {       // first pass of the per-row formats: the row's range
      float neglo, hi;
      group_range(P, cbits, neglo, hi);
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {          // (all 32 lanes hold groups of the same row; dead lanes hold zeros)
        neglo = fmaxf(neglo, __shfl_xor_sync(0xFFFFFFFFu, neglo, d));
        hi = fmaxf(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, d));
      }
      if (lane == 0) {
        atomicMax(p.rowstats + 2 * row, __float_as_uint(neglo));
        atomicMax(p.rowstats + 2 * row + 1, __float_as_uint(hi));
      }
      continue;
    }
    if (!full) {                                   // the statistics only
      if (p.mse) {
        const float e = rq::group_error(P, cbits, p.format);
        if (live) p.mse[row * ng + g] = e;
      } else {
        const uint32_t sb = rq::group_scale_byte(P, cbits);
        if (live) p.scale_bytes[row * ng + g] = (uint8_t)sb;
      }
      continue;
    }
    float out[32];
    if (p.format == kFormatNone) {                 // the rotation itself
      const uint64_t cc = rq::pack2(__uint_as_float(cbits), __uint_as_float(cbits));
#pragma unroll
      for (int k = 0; k < 16; ++k) rq::unpack2(rq::mul2(P[k], cc), out[2 * k], out[2 * k + 1]);
    } else if (p.format >= kFormatRowSym) {
      const float neglo = __uint_as_float(__ldcg(p.rowstats + 2 * row));
      const float hi = __uint_as_float(__ldcg(p.rowstats + 2 * row + 1));
      row_dequant(P, cbits, p.format == kFormatRowAsym, neglo, hi, out);
    } else {
      group_dequant(P, cbits, p.format, out);
    }
    // lane l -> buffer row l (128 bytes), piece j at position j ^ (l & 7)
    __syncwarp();                                  // the previous task's reads of the buffer are done
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<float4*>(wbuf + lane * 32 + ((j ^ (lane & 7)) << 2)) =
          make_float4(out[4 * j], out[4 * j + 1], out[4 * j + 2], out[4 * j + 3]);
    __syncwarp();
    // instruction i writes groups 4i .. 4i+3 of the chunk: 8 lanes per group, 16 bytes each
    const int gbase = g - lane;
    float* rowp = p.deq + row * p.ldd + (int64_t)gbase * 32;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = i * 4 + (lane >> 3), c = lane & 7;
      const float4 v = *reinterpret_cast<const float4*>(wbuf + r * 32 + ((c ^ (r & 7)) << 2));
      if (gbase + r < ng) *reinterpret_cast<float4*>(rowp + r * 32 + c * 4) = v;
    }
  }
}

// block: 1 (identity), 2, 4, 8, 16, 32, 64 or 128.  Exactly one of deq / mse / scale_bytes is set — or none of
// them and rowstats, for the first pass of the per-row formats.
inline bro_status launch(const void* x, int64_t M, int64_t K, int64_t ldx, int block, const void* signs, int format,
                         float* deq, int64_t ldd, float* mse, uint8_t* scale_bytes, int sm_count, cudaStream_t st,
                         uint32_t* rowstats = nullptr) {
  Params p;
  p.rowstats = rowstats;
  p.x = static_cast<const uint16_t*>(x);
  p.M = M; p.K = K; p.ldx = ldx;
  p.signs = static_cast<const uint16_t*>(signs);
  p.deq = deq;
  p.ldd = ldd;
  p.mse = mse;
  p.scale_bytes = scale_bytes;
  p.format = format;
  p.chunks_per_row = (int)((K / 32 + 31) / 32);
  p.total_tasks = M * p.chunks_per_row;
  const int64_t want = (p.total_tasks + kWarps - 1) / kWarps;
  const int64_t cap = (int64_t)sm_count * 8;
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  auto go = [&](auto kernel) -> bro_status {
    return cuda_ok(launch_kernel(kernel, grid, kThreads, 0, st, 1, p), "fake_quantize launch") ? BRO_OK : BRO_ERR_CUDA;
  };
  int lg = 0;
  while ((1 << lg) < block) ++lg;
  // (with the identity the signs only flip the output signs; they are applied all the same)
  if (signs) {
    switch (lg) {
      case 0: return go(fake_quantize_kernel<0, true>);
      case 1: return go(fake_quantize_kernel<1, true>);
      case 2: return go(fake_quantize_kernel<2, true>);
      case 3: return go(fake_quantize_kernel<3, true>);
      case 4: return go(fake_quantize_kernel<4, true>);
      case 5: return go(fake_quantize_kernel<5, true>);
      case 6: return go(fake_quantize_kernel<6, true>);
      default: return go(fake_quantize_kernel<7, true>);
    }
  }
  switch (lg) {
    case 0: return go(fake_quantize_kernel<0, false>);
    case 1: return go(fake_quantize_kernel<1, false>);
    case 2: return go(fake_quantize_kernel<2, false>);
    case 3: return go(fake_quantize_kernel<3, false>);
    case 4: return go(fake_quantize_kernel<4, false>);
    case 5: return go(fake_quantize_kernel<5, false>);
    case 6: return go(fake_quantize_kernel<6, false>);
    default: return go(fake_quantize_kernel<7, false>);
  }
}

}  // namespace fq
}  // namespace bro
