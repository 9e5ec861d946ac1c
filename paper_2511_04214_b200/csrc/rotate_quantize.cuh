// Kernel 1: fused block-Hadamard rotation + MXFP4 quantisation (paper Sec. 4.3 Eq. 1, Sec. 4.1).
//
// HBM-bound streaming kernel: 2 bytes in and 0.53125 bytes out per element, one pass.
//
//  * One persistent CTA per SM.  A producer thread streams 128-row x 128-column bf16 tiles into
//    a ring of shared-memory stages with TMA (two 128x64 boxes per tile, 128-byte swizzle), so
//    the loads in flight are bounded by shared memory, not by registers.
//  * 16 consumer warps.  Each thread owns one whole MX group (32 consecutive channels of one
//    row): four conflict-free 16-byte shared loads, then the 5 butterfly stages of the 32-point
//    Walsh-Hadamard transform entirely in registers — no shuffles for block = 32.  Blocks of 64
//    and 128 add one or two cross-lane stages (the 2 or 4 groups of a block sit in lanes that
//    differ in bit 0 / bit 3).
//  * fp32 arithmetic in exactly this order: butterflies (a+b, a-b) with ascending stride, one
//    multiply by c = fp32(1/sqrt(block)), amax over the group, shared exponent
//    E = max(expfield(amax) - 2, 0) - 127, r = y * 2^-E, round-to-nearest-even to E2M1 with
//    saturation.  The multiply by c and the exact scaling by 2^-E are merged into one multiply by
//    c*2^-E whenever that product is a normal fp32 (bit-identical result); otherwise the two
//    multiplies are done separately.
//  * Output: one 16-byte store of 32 packed codes per thread; the 4 scale bytes of a row inside
//    the tile are gathered with two shuffles and written as one 32-bit store.
#pragma once

#include <cuda_fp16.h>

#include "bro_common.cuh"

namespace bro {
namespace rq {

constexpr int kTileRows = 128;
constexpr int kTileCols = 128;              // 4 MX groups
constexpr int kBoxCols = 64;                // one TMA box: 128 rows x 64 bf16 = 128 B per row
constexpr int kBoxBytes = kTileRows * kBoxCols * 2;   // 16 KiB
constexpr int kStageBytes = 2 * kBoxBytes;            // 32 KiB
constexpr int kStages = 6;
constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;   // + 1 producer warp
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;

struct Params {
  int64_t M, K;
  int64_t tiles_m, tiles_k;     // tiles_k covers the scale padding when layout == GEMM
  uint8_t* codes;               // [M, K/2]
  uint8_t* scales;
  int64_t scale_kblocks;        // GEMM layout: 512-byte blocks per 128-row block
  int layout;                   // bro_layout
  const uint16_t* signs;        // [K] bf16 +-1 (randomised rotation, kernels with SIGNS) or nullptr
};

// x diag(s): flip the bf16 sign bits of a 16-byte chunk of x where the sign vector is negative.
// One three-input logic operation per 32-bit word (x ^ (s & 0x80008000)); exact.
__device__ __forceinline__ uint4 apply_signs(uint4 q, uint4 sg) {
  q.x ^= sg.x & 0x80008000u;
  q.y ^= sg.y & 0x80008000u;
  q.z ^= sg.z & 0x80008000u;
  q.w ^= sg.w & 0x80008000u;
  return q;
}

__device__ __forceinline__ uint32_t pack_e2m1x8(float r0, float r1, float r2, float r3, float r4,
                                                float r5, float r6, float r7) {
  // cvt.rn.satfinite.e2m1x2.f32 d, a, b : a -> bits 4..7, b -> bits 0..3 (nearest even, +-6 clamp)
  uint32_t w;
  asm("{ .reg .b8 b0, b1, b2, b3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
      "mov.b32 %0, {b0, b1, b2, b3}; }"
      : "=r"(w)
      : "f"(r0), "f"(r1), "f"(r2), "f"(r3), "f"(r4), "f"(r5), "f"(r6), "f"(r7));
  return w;
}

// c = fp32 nearest 1/sqrt(2^LOG2B)
template <int LOG2B>
__device__ __forceinline__ constexpr uint32_t norm_bits() {
  // even exponent: exact power of two; odd: fp32(sqrt 2) = 0x3FB504F3 scaled by a power of two
  return (LOG2B % 2 == 0) ? (uint32_t)(127 - LOG2B / 2) << 23
                          : 0x3FB504F3u - ((uint32_t)((LOG2B + 1) / 2) << 23);
}

// ---- packed fp32x2 arithmetic (sm_100): one issue slot for two IEEE round-to-nearest results.
// A group's 32 values live in 16 register pairs; pair k holds elements (2k, 2k+1).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t shfl_xor2(uint64_t v, int lane_mask) {
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
  lo = __shfl_xor_sync(0xFFFFFFFFu, lo, lane_mask);
  hi = __shfl_xor_sync(0xFFFFFFFFu, hi, lane_mask);
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}

// 8 bf16 (one 16-byte chunk) -> 4 pairs, fused with butterfly stage h = 1, which pairs the two
// halves of one 32-bit word: (lo, hi) -> (lo + hi, lo - hi).
__device__ __forceinline__ void unpack_stage1(const uint4& q, uint64_t* P) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float lo = __uint_as_float(w[k] << 16);
    const float hi = __uint_as_float(w[k] & 0xFFFF0000u);
    P[k] = pack2(__fadd_rn(lo, hi), __fsub_rn(lo, hi));
  }
}

// Butterfly stages h = 2, 4, 8, 16 on pairs (ascending stride): pair k meets pair k ^ (h/2).
__device__ __forceinline__ void fwht32_stages_2_to_16(uint64_t (&P)[16]) {
#pragma unroll
  for (int hp = 1; hp < 16; hp <<= 1) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((k & hp) == 0) {
        const uint64_t a = P[k], b = P[k + hp];
        P[k] = add2(a, b);
        P[k + hp] = sub2(a, b);
      }
    }
  }
}

// The same for a rotation inside the MX group (blocks of 2..16 channels: LOG2B = 1..4): the stages of
// stride 2 .. B/2 only (stage h = 1 is in unpack_stage1).
template <int LOG2B>
__device__ __forceinline__ void fwht32_stages_below(uint64_t (&P)[16]) {
  static_assert(LOG2B >= 1 && LOG2B <= 4, "blocks of 2..16");
#pragma unroll
  for (int hp = 1; hp < (1 << (LOG2B - 1)); hp <<= 1) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((k & hp) == 0) {
        const uint64_t a = P[k], b = P[k + hp];
        P[k] = add2(a, b);
        P[k + hp] = sub2(a, b);
      }
    }
  }
}

// ---- blocks of 64 / 128 channels: cross-lane stages that exchange HALF of each lane's values --------
// The 2 (or 4) MX groups of a block sit in neighbouring lanes.  A butterfly stage between two lanes
// needs, for every element i, a + b in one lane and a - b in the other.  Instead of every lane
// fetching all 32 partner values and producing 32 results, each lane keeps 16 of its values, sends
// the other 16, and produces BOTH the sum and the difference for the 16 elements it kept: half the
// shuffles, and the arithmetic stays on packed pairs.  Afterwards a lane holds 16 values of one output
// group and 16 values of another (two 8-byte code stores instead of one 16-byte store; the group
// maximum takes one more shuffle).
//
// So that both lanes of a pair run the same instructions on the same registers, the odd lane loads
// its 64 bytes with the two 32-byte halves exchanged (register pair k holds true pair k ^ 8): every
// lane then keeps registers 0..7 and sends registers 8..15.  Stages h = 1..8 never cross the halves;
// stage h = 16 does, and is written as two fused multiply-adds with the lane's sign s (+1 even lane,
// -1 odd lane), which yields a + b and a - b in the registers where this lane expects them:
//   P'[k]   = s * P[k]   + P[k+8]      P'[k+8] = -s * P[k+8] + P[k]
// Each is ONE rounding of the exact sum or difference (a product with +-1 is exact), i.e. bit-identical
// to the add / subtract of the contract, including the sign of an exact zero (x - y == x + (-y)).
__device__ __forceinline__ void fwht32_stages_2_to_8(uint64_t (&P)[16]) {
#pragma unroll
  for (int hp = 1; hp < 8; hp <<= 1) {
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((k & hp) == 0) {
        const uint64_t a = P[k], b = P[k + hp];
        P[k] = add2(a, b);
        P[k + hp] = sub2(a, b);
      }
    }
  }
}
__device__ __forceinline__ void stage16_halves_exchanged(uint64_t (&P)[16], uint64_t s2, uint64_t ns2) {
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint64_t a = P[k], b = P[k + 8];
    P[k] = fma2(a, s2, b);
    P[k + 8] = fma2(b, ns2, a);
  }
}

// amax of the 16 values held in 8 pairs (three-input maximum of absolute values, two chains).
__device__ __forceinline__ float amax_pairs8(const uint64_t (&P)[8]) {
  float m = 0.f, m2 = 0.f;
#pragma unroll
  for (int k = 0; k < 8; k += 2) {
    float lo, hi, lo2, hi2;
    unpack2(P[k], lo, hi);
    unpack2(P[k + 1], lo2, hi2);
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m) : "f"(lo), "f"(hi));
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m2) : "f"(lo2), "f"(hi2));
  }
  return fmaxf(m, m2);
}
// Scale byte of a group from its pre-normalisation amax, and the 16 codes of the half group in P
// (same arithmetic as quantize_group).
__device__ __forceinline__ uint32_t encode_pairs8(const uint64_t (&P)[8], float amax, uint32_t cbits, uint32_t (&w)[2]) {
  const float c = __uint_as_float(cbits);
  const uint32_t ef = __float_as_uint(__fmul_rn(amax, c)) >> 23;
  const uint32_t s = ef > 2u ? ef - 2u : 0u;
  float r[16];
  if (ef >= 27u && ef <= 250u) {
    const float c2 = __uint_as_float(cbits + ((127u - s) << 23));
    const uint64_t cc = pack2(c2, c2);
#pragma unroll
    for (int k = 0; k < 8; ++k) unpack2(mul2(P[k], cc), r[2 * k], r[2 * k + 1]);
  } else {
    const float p2 = __uint_as_float((254u - s) << 23);
    const uint64_t cc = pack2(c, c), pp = pack2(p2, p2);
#pragma unroll
    for (int k = 0; k < 8; ++k) unpack2(mul2(mul2(P[k], cc), pp), r[2 * k], r[2 * k + 1]);
  }
#pragma unroll
  for (int j = 0; j < 2; ++j)
    w[j] = pack_e2m1x8(r[8 * j], r[8 * j + 1], r[8 * j + 2], r[8 * j + 3], r[8 * j + 4], r[8 * j + 5],
                       r[8 * j + 6], r[8 * j + 7]);
  return s;
}

// The cross-lane stages of a 64- or 128-channel block on the registers described above, then the
// quantisation of the two half groups this lane ends up with.
//   lane & 1   which 16 elements of a group this lane keeps (0: elements 0..15, 1: 16..31)
//   lane & 2   (blocks of 128) which pair of groups: 0 -> groups 0 / 2 of the block, 1 -> groups 1 / 3
// Outputs: wx / sx = codes of this lane's 16 elements and scale byte of group X, wy / sy of group Y, with
//   block 64 : X = group 0, Y = group 1 of the block;   block 128 : X = group (lane>>1)&1, Y = X + 2.
// P must hold the values after stages h = 1..8 (odd lanes: halves exchanged).
template <int LOG2B>
__device__ __forceinline__ void cross_lane_split(uint64_t (&P)[16], int lane, uint32_t cbits, uint32_t (&wx)[2],
                                                 uint32_t& sx, uint32_t (&wy)[2], uint32_t& sy) {
  static_assert(LOG2B == 6 || LOG2B == 7, "blocks of 64 or 128 channels");
  const float s0 = (lane & 1) ? -1.f : 1.f;
  const uint64_t s0p = pack2(s0, s0), ns0p = pack2(-s0, -s0);
  stage16_halves_exchanged(P, s0p, ns0p);
  uint64_t X[8], Y[8];
  if (LOG2B == 6) {
    // stage h = 32 with lane ^ 1: kept K = P[0..7], received R = partner's P[8..15] (the same elements)
    //   even lane: X = K + R, Y = K - R;   odd lane: X = R + K, Y = R - K
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const uint64_t R = shfl_xor2(P[8 + k], 1);
      X[k] = add2(P[k], R);
      Y[k] = fma2(P[k], s0p, mul2(R, ns0p));
    }
  } else {
    // stage h = 32 with lane ^ 1, written so that lanes of the second group pair (lane & 2) get sum and
    // difference in exchanged registers: they keep the difference and send the sum in stage h = 64.
    const bool second = (lane & 2) != 0;
    const float one = 1.f;
    const uint64_t c1 = second ? s0p : pack2(one, one), c2 = second ? ns0p : pack2(one, one);
    const uint64_t c3 = second ? pack2(one, one) : s0p, c4 = second ? pack2(one, one) : ns0p;
    const float s1 = second ? -1.f : 1.f;
    const uint64_t s1p = pack2(s1, s1), ns1p = pack2(-s1, -s1);
    uint64_t U[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const uint64_t R = shfl_xor2(P[8 + k], 1);
      U[k] = fma2(P[k], c1, mul2(R, c2));            // kept for stage h = 64
      const uint64_t V = fma2(P[k], c3, mul2(R, c4)); // sent
      const uint64_t R2 = shfl_xor2(V, 2);
      X[k] = add2(U[k], R2);
      Y[k] = fma2(U[k], s1p, mul2(R2, ns1p));
    }
  }
  float mx = amax_pairs8(X), my = amax_pairs8(Y);
  mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
  my = fmaxf(my, __shfl_xor_sync(0xFFFFFFFFu, my, 1));
  sx = encode_pairs8(X, mx, cbits, wx);
  sy = encode_pairs8(Y, my, cbits, wy);
}

// One butterfly stage across two lanes that hold the low / high half of the pairs.
// low lane: a + b ; high lane: a - b = own * (-1) + other (exact, one rounding).
__device__ __forceinline__ void cross_lane_stage(uint64_t (&P)[16], int lane_mask, bool is_high) {
  const float sgn = is_high ? -1.f : 1.f;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float lo, hi;
    unpack2(P[k], lo, hi);
    const float olo = __shfl_xor_sync(0xFFFFFFFFu, lo, lane_mask);
    const float ohi = __shfl_xor_sync(0xFFFFFFFFu, hi, lane_mask);
    P[k] = pack2(__fmaf_rn(lo, sgn, olo), __fmaf_rn(hi, sgn, ohi));
  }
}

// Quantise the 32 fp32 values held in P (pre-normalisation: y = v*c) of one MX group.
// Returns the scale byte; writes 4 code words.
__device__ __forceinline__ uint32_t quantize_group(const uint64_t (&P)[16], uint32_t cbits, uint32_t (&w)[4]) {
  // amax with the three-input maximum of absolute values (one instruction per pair); two
  // accumulators halve the dependent chain
  float m = 0.f, m2 = 0.f;
#pragma unroll
  for (int k = 0; k < 16; k += 2) {
    float lo, hi, lo2, hi2;
    unpack2(P[k], lo, hi);
    unpack2(P[k + 1], lo2, hi2);
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m) : "f"(lo), "f"(hi));
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m2) : "f"(lo2), "f"(hi2));
  }
  m = fmaxf(m, m2);
  const float c = __uint_as_float(cbits);
  // amax of y: rounding is monotonic, so max_i fl(|v_i| c) = fl(max_i |v_i| * c)
  const uint32_t ef = __float_as_uint(__fmul_rn(m, c)) >> 23;
  const uint32_t s = ef > 2u ? ef - 2u : 0u;
  float r[32];
  if (ef >= 27u && ef <= 250u) {
    // c * 2^-E is a normal fp32: one multiply, bit-identical to (v*c)*2^-E
    const float c2 = __uint_as_float(cbits + ((127u - s) << 23));
    const uint64_t cc = pack2(c2, c2);
#pragma unroll
    for (int k = 0; k < 16; ++k) unpack2(mul2(P[k], cc), r[2 * k], r[2 * k + 1]);
  } else {
    const float p2 = __uint_as_float((254u - s) << 23);   // 2^-E, E = s - 127
    const uint64_t cc = pack2(c, c), pp = pack2(p2, p2);
#pragma unroll
    for (int k = 0; k < 16; ++k) unpack2(mul2(mul2(P[k], cc), pp), r[2 * k], r[2 * k + 1]);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j)
    w[j] = pack_e2m1x8(r[8 * j], r[8 * j + 1], r[8 * j + 2], r[8 * j + 3], r[8 * j + 4], r[8 * j + 5],
                       r[8 * j + 6], r[8 * j + 7]);
  return s;
}

// Scale byte only: the E8M0 byte quantize_group would assign to the group held in P.
constexpr int kFormatScaleOnly = 4;     // `format` value of the analysis kernels that selects this output
__device__ __forceinline__ uint32_t group_scale_byte(const uint64_t (&P)[16], uint32_t cbits) {
  float m = 0.f, m2 = 0.f;
#pragma unroll
  for (int k = 0; k < 16; k += 2) {
    float lo, hi, lo2, hi2;
    unpack2(P[k], lo, hi);
    unpack2(P[k + 1], lo2, hi2);
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m) : "f"(lo), "f"(hi));
    asm("max.abs.f32 %0, %0, %1, %2;" : "+f"(m2) : "f"(lo2), "f"(hi2));
  }
  m = fmaxf(m, m2);
  const uint32_t ef = __float_as_uint(__fmul_rn(m, __uint_as_float(cbits))) >> 23;
  return ef > 2u ? ef - 2u : 0u;
}

// Quantisation error of one group of 32 (paper Sec. 4.1-4.2: block-level error under the shared
// scale; Sec. 3.2 / Fig. 2-3 for the formats compared): mean over the group of (y - deq(Q(y)))^2 with
// y = v * c the rotated values.  `format`: 0 MXFP4 (E2M1, scale 2^E, E = floor(log2 amax) - 2),
// 1 BFP4 (E2M1, scale fp16(amax / 6)), 2 MXINT4 (k/4 with |k| <= 7, scale 2^floor(log2 amax)),
// 3 BINT4 (|k| <= 7, scale fp16(amax / 7)); round to nearest even, saturating.
// E2M1 codes come from the same conversion instruction as in quantize_group and are decoded again
// in hardware (e2m1x2 -> f16x2).  With a power-of-two scale the difference is exact in the scaled
// domain; with an fp16 scale it is one fused multiply-add.  Squares and their sum are fp32.
__device__ __forceinline__ float group_error(const uint64_t (&P)[16], uint32_t cbits, int format) {
  const float c = __uint_as_float(cbits);
  const uint64_t cc = pack2(c, c);
  float y[32];
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    unpack2(mul2(P[k], cc), y[2 * k], y[2 * k + 1]);
    y[2 * k] = fabsf(y[2 * k]);             // every format is symmetric: work on magnitudes
    y[2 * k + 1] = fabsf(y[2 * k + 1]);
  }
  float m = 0.f;
#pragma unroll
  for (int i = 0; i < 32; ++i) m = fmaxf(m, y[i]);
  const uint32_t ef = __float_as_uint(m) >> 23;
  auto e2m1 = [](float r0, float r1, float& q0, float& q1) {
    uint32_t h;
    asm("{ .reg .b8 b; cvt.rn.satfinite.e2m1x2.f32 b, %2, %1; cvt.rn.f16x2.e2m1x2 %0, b; }" : "=r"(h) : "f"(r0), "f"(r1));
    q0 = __half2float(__ushort_as_half((unsigned short)(h & 0xFFFFu)));
    q1 = __half2float(__ushort_as_half((unsigned short)(h >> 16)));
  };
  float acc = 0.f;
  if (format == 0 || format == 2) {
    const uint32_t s = format == 0 ? (ef > 2u ? ef - 2u : 0u) : ef;
    const float inv = __uint_as_float(s <= 253u ? ((254u - s) << 23) : 0x00400000u);   // 2^-E, E = s - 127 (2^-127 is subnormal)
    const float pe = __uint_as_float(s >= 1u ? (s << 23) : 0x00400000u);    // 2^E (2^-127 is subnormal)
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
      const float r0 = __fmul_rn(y[i], inv), r1 = __fmul_rn(y[i + 1], inv);
      float q0, q1;
      if (format == 0) {
        e2m1(r0, r1, q0, q1);
      } else {
        q0 = 0.25f * (float)min(__float2int_rn(__fmul_rn(r0, 4.f)), 7);
        q1 = 0.25f * (float)min(__float2int_rn(__fmul_rn(r1, 4.f)), 7);
      }
      const float d0 = __fsub_rn(r0, q0), d1 = __fsub_rn(r1, q1);
      acc = __fadd_rn(acc, __fmul_rn(d0, d0));
      acc = __fadd_rn(acc, __fmul_rn(d1, d1));
    }
    return __fmul_rn(__fmul_rn(__fmul_rn(acc, 0.03125f), pe), pe);
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
    float q0 = 0.f, q1 = 0.f;
    if (sc != 0.f) {
      const float r0 = __fdiv_rn(y[i], sc), r1 = __fdiv_rn(y[i + 1], sc);
      if (format == 1) {
        e2m1(r0, r1, q0, q1);
      } else {
        q0 = (float)min(__float2int_rn(r0), 7);
        q1 = (float)min(__float2int_rn(r1), 7);
      }
    }
    const float d0 = __fmaf_rn(-q0, sc, y[i]), d1 = __fmaf_rn(-q1, sc, y[i + 1]);
    acc = __fadd_rn(acc, __fmul_rn(d0, d0));
    acc = __fadd_rn(acc, __fmul_rn(d1, d1));
  }
  return __fmul_rn(acc, 0.03125f);
}

// SIGNS: the randomised rotation R_i = diag(s) H / sqrt(block) (paper Sec. 5.1) — the channel signs
// are applied to the bf16 inputs as they leave shared memory; everything else is unchanged.
template <int LOG2B, bool SIGNS>
__global__ void __launch_bounds__(kThreads, 1)
rotate_quantize_kernel(const __grid_constant__ CUtensorMap tmx, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzle needs 1 KiB
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  // full[s] at bar_base + 8*s ; empty[s] at bar_base + 8*(kStages + s)
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_base + 8 * s, 1);
      mbar_init(bar_base + 8 * (kStages + s), kConsumerWarps);
    }
    mbar_fence_init();
    fence_proxy_async_smem();
  }
  __syncthreads();
  griddep_wait();               // x may be written, codes/scales still read, by the kernel before
  // (only now: a dependent that starts early may then rely on everything older than this kernel)
  griddep_launch_dependents();

  const int64_t total_tiles = p.tiles_m * p.tiles_k;

  if (warp == kConsumerWarps) {
    // ---------------- producer ----------------
    if (lane == 0) {
      tma_prefetch_desc(&tmx);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int64_t issued = 0;
      const int tiles_k = (int)p.tiles_k;
      int tm = (int)(blockIdx.x / (unsigned)tiles_k), tk = (int)(blockIdx.x % (unsigned)tiles_k);
      const int step_m = (int)(gridDim.x / (unsigned)tiles_k), step_k = (int)(gridDim.x % (unsigned)tiles_k);
      for (int64_t t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        if (issued >= kStages)
          ok = mbar_wait(bar_base + 8 * (kStages + stage), phase ^ 1u, SITE_RQ_EMPTY);
        if (!ok) break;
        const uint32_t full = bar_base + 8 * stage;
        const uint32_t dst = smem_base + stage * kStageBytes;
        mbar_arrive_expect_tx(full, kStageBytes);
        tma_load_2d(dst, &tmx, tk * kTileCols, tm * kTileRows, full);
        tma_load_2d(dst + kBoxBytes, &tmx, tk * kTileCols + kBoxCols, tm * kTileRows, full);
        ++issued;
        if (++stage == kStages) { stage = 0; phase ^= 1u; }
        tm += step_m;
        tk += step_k;
        if (tk >= tiles_k) { tk -= tiles_k; ++tm; }
      }
      if (!ok) {
        // A consumer gave up.  Do not leave the CTA while copies may still land in its shared
        // memory: wait (bounded) for the last load armed on every stage.  Issue i used stage
        // i % kStages in phase (i / kStages) & 1.
        const int64_t first = issued > kStages ? issued - kStages : 0;
        for (int64_t i = first; i < issued; ++i)
          mbar_wait(bar_base + 8 * (int)(i % kStages), (uint32_t)((i / kStages) & 1), SITE_RQ_DRAIN);
      }
    }
  } else {
    // ---------------- consumers ----------------
    const int gg = lane & 1;                 // group within the 64-column box
    const int box = (lane >> 3) & 1;         // which box of the tile
    const int row = warp * 8 + ((lane >> 4) << 2) + ((lane >> 1) & 3);   // row within the tile
    const int g = box * 2 + gg;              // group within the tile (0..3)
    // 16-byte chunk j of this group sits at chunk index (gg*4 + j) ^ (row & 7) of its 128-B row
    const uint32_t row_off = (uint32_t)box * kBoxBytes + (uint32_t)row * 128u;
    const uint32_t sw = (uint32_t)(row & 7);
    constexpr uint32_t cbits = norm_bits<LOG2B>();

    int stage = 0;
    uint32_t phase = 0;
    const int tiles_k = (int)p.tiles_k;
    int tm = (int)(blockIdx.x / (unsigned)tiles_k), tk = (int)(blockIdx.x % (unsigned)tiles_k);
    const int step_m = (int)(gridDim.x / (unsigned)tiles_k), step_k = (int)(gridDim.x % (unsigned)tiles_k);
    for (int64_t t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      if (!mbar_wait(bar_base + 8 * stage, phase, SITE_RQ_FULL)) break;
      const uint32_t src = smem_base + stage * kStageBytes + row_off;
      uint64_t P[16];
      uint4 sg[4] = {};
      if (SIGNS && (tk * (kTileCols / 32) + g) * 32 < (int)p.K) {
        const uint4* sp = reinterpret_cast<const uint4*>(p.signs + (tk * kTileCols + g * 32));
#pragma unroll
        for (int j = 0; j < 4; ++j) sg[j] = __ldg(sp + j);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint4 q = lds128(src + ((((uint32_t)gg * 4u + j) ^ sw) << 4));
        if (SIGNS) q = apply_signs(q, sg[j]);
        unpack_stage1(q, P + 4 * j);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_base + 8 * (kStages + stage));
      if (++stage == kStages) { stage = 0; phase ^= 1u; }

      fwht32_stages_2_to_16(P);
      if (LOG2B >= 6) cross_lane_stage(P, 1, gg != 0);
      if (LOG2B >= 7) cross_lane_stage(P, 8, box != 0);

      uint32_t w[4];
      const uint32_t s = quantize_group(P, cbits, w);

      const int64_t grow = (int64_t)tm * kTileRows + row;
      const int ggrp = tk * (kTileCols / 32) + g;         // group index along K
      const bool in_k = ggrp * 32 < (int)p.K;
      if (grow < p.M && in_k) {
        uint4* dst = reinterpret_cast<uint4*>(p.codes + grow * (p.K >> 1) + ggrp * 16);
        *dst = make_uint4(w[0], w[1], w[2], w[3]);
      }
      // gather the row's 4 scale bytes of this tile into the lane with gg == 0 && box == 0
      uint32_t sb = in_k ? s : 0u;
      sb |= __shfl_xor_sync(0xFFFFFFFFu, sb, 1) << 8;
      sb |= __shfl_xor_sync(0xFFFFFFFFu, sb, 8) << 16;
      if (g == 0) {
        if (p.layout == BRO_LAYOUT_GEMM) {
          // 512-byte block (tm, tk): byte (r%32)*16 + (r/32)*4 + g ; padding rows included
          const int64_t off = ((int64_t)tm * p.scale_kblocks + tk) * 512 + (row & 31) * 16 + (row >> 5) * 4;
          *reinterpret_cast<uint32_t*>(p.scales + off) = sb;
        } else if (grow < p.M) {
          const int ng = (int)(p.K >> 5);
          uint8_t* dst = p.scales + grow * ng + tk * 4;
          if (tk * 4 + 4 <= ng && ((reinterpret_cast<uintptr_t>(dst) & 3) == 0)) {
            *reinterpret_cast<uint32_t*>(dst) = sb;
          } else {
            for (int i = 0; i < 4 && tk * 4 + i < ng; ++i) dst[i] = (uint8_t)(sb >> (8 * i));
          }
        }
      }
      tm += step_m;
      tk += step_k;
      if (tk >= tiles_k) { tk -= tiles_k; ++tm; }
    }
  }
}

}  // namespace rq
}  // namespace bro
