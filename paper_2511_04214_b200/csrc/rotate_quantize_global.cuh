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
    if (p.format == rq::kFormatScaleOnly) {   // analysis mode (uniform over the grid): scale byte only
      const uint32_t sbyte = rq::group_scale_byte(P, cbits);
      if (live) p.scales[row * (p.K >> 5) + gi] = (uint8_t)sbyte;
      continue;
    }
    if (p.mse) {                 // analysis mode (uniform over the grid)
      const float e = rq::group_error(P, cbits, p.format);
      if (live) p.mse[row * (p.K >> 5) + gi] = e;
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

inline bro_status launch(const void* x, int64_t M, int64_t K, int64_t ldx, const void* signs, void* codes,
                         void* scales, float* mse, int format, bro_layout layout, int64_t scale_kblocks, int sm_count, cudaStream_t st) {
  Params p;
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
  if (layout == BRO_LAYOUT_GEMM && !mse && format != rq::kFormatScaleOnly) {
    // padding rows / groups of the tiled scale buffer must read as 0
    const size_t bytes = (size_t)((M + 127) / 128) * (size_t)scale_kblocks * 512;
    if (cudaMemsetAsync(scales, 0, bytes, st) != cudaSuccess) return BRO_ERR_CUDA;
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
