// libbro: C ABI over the two sm_100a kernels (see include/bro.h for the contract).
// Host-side work only: argument validation, TMA tensor-map encoding, launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/bro.h"
#include "bro_common.cuh"
#include "rotate_quantize.cuh"
#include "rotate_quantize_global.cuh"
#include "rotate_quantize_direct.cuh"
#include "gemm_mxfp4.cuh"
#include "gemm_mxfp4_2cta.cuh"
#include "scale_stats.cuh"
#include "fake_quantize.cuh"

namespace {

using bro::rq::Params;

constexpr int64_t kGroup = 32;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }
inline int log2_of(int64_t v) {
  int lg = 0;
  while (((int64_t)1 << lg) < v) ++lg;
  return lg;
}

// ---- device / driver plumbing ------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

struct DeviceInfo {
  bool ok = false;
  int sm_count = 0;
};

// Per-device facts, looked up once per device.
bro_status device_info(DeviceInfo* out) {
  static DeviceInfo cache[64];
  static bool known[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return BRO_ERR_CUDA;
  if (dev < 0 || dev >= 64) return BRO_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(mu);
  if (!known[dev]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return BRO_ERR_CUDA;
    cache[dev].ok = (prop.major == 10);
    cache[dev].sm_count = prop.multiProcessorCount;
    known[dev] = true;
  }
  *out = cache[dev];
  return out->ok ? BRO_OK : BRO_ERR_ARCH;
}

// 2-D row-major tensor map: dims {inner, rows}, row pitch in bytes, box {box_inner, box_rows}.
bro_status make_map_2d(CUtensorMap* map, CUtensorMapDataType dt, size_t elem_bytes, const void* base,
                       uint64_t inner, uint64_t rows, uint64_t pitch_bytes, uint32_t box_inner,
                       uint32_t box_rows, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) {
    snprintf(bro::g_last_cuda_error, sizeof(bro::g_last_cuda_error), "cuTensorMapEncodeTiled unavailable");
    return BRO_ERR_CUDA;
  }
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  (void)elem_bytes;
  CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    snprintf(bro::g_last_cuda_error, sizeof(bro::g_last_cuda_error), "cuTensorMapEncodeTiled: CUresult %d", (int)r);
  return r == CUDA_SUCCESS ? BRO_OK : BRO_ERR_CUDA;
}

template <typename K>
bro_status set_smem(K kernel, int bytes) {
  return bro::cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes),
                      "cudaFuncSetAttribute")
             ? BRO_OK
             : BRO_ERR_CUDA;
}

int64_t gemm_scale_kblocks(int64_t K) { return 2 * ceil_div(K, 256); }

}  // namespace

// Packed 4-bit codes viewed as bytes: [rows, K/2], box = 128 bytes x box_rows, 128-byte swizzle.
bro_status bro::gemm::make_codes_map(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int box_rows) {
  return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base, (uint64_t)(K / 2), (uint64_t)rows,
                     (uint64_t)(K / 2), 128, (uint32_t)box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

// bf16 output [M, ldy]: box = 64 columns (128 bytes) x 32 rows (what one epilogue warp stores at a
// time), 128-byte swizzle to match its staging buffer.
bro_status bro::gemm::make_out_map(CUtensorMap* map, const void* y, int64_t M, int64_t N, int64_t ldy) {
  return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy * 2,
                     2 * bro::gemm::kChunkCols, 32, CU_TENSOR_MAP_SWIZZLE_128B);
}

// Scale tensor in the tensor-core layout viewed as 32-bit words: one row per 128-row block
// (kblocks * 512 bytes), box = one K step (1024 bytes) x box_rows row blocks, no swizzle.
bro_status bro::gemm2::make_scale_map(CUtensorMap* map, const void* scales, int64_t rows, int64_t kblocks,
                                      int box_rows) {
  return make_map_2d(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, scales, (uint64_t)(kblocks * 128),
                     (uint64_t)ceil_div(rows, 128), (uint64_t)(kblocks * 512), 256, (uint32_t)box_rows,
                     CU_TENSOR_MAP_SWIZZLE_NONE);
}

// Rows of x as a 3-D tensor {64 bf16, K / 64, M} with strides {128 bytes, ldx * 2 bytes}: a box of
// whole rows lands in shared memory as 128-byte segments with the 128-byte swizzle.
bro_status bro::rqg::make_row_map(CUtensorMap* map, const void* x, int64_t M, int64_t K, int64_t ldx, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) {
    snprintf(bro::g_last_cuda_error, sizeof(bro::g_last_cuda_error), "cuTensorMapEncodeTiled unavailable");
    return BRO_ERR_CUDA;
  }
  cuuint64_t dims[3] = {64, (cuuint64_t)(K / 64), (cuuint64_t)M};
  cuuint64_t strides[2] = {128, (cuuint64_t)ldx * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)(K / 64), (cuuint32_t)box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    snprintf(bro::g_last_cuda_error, sizeof(bro::g_last_cuda_error), "cuTensorMapEncodeTiled (rows): CUresult %d", (int)r);
  return r == CUDA_SUCCESS ? BRO_OK : BRO_ERR_CUDA;
}

namespace {

// One warp waits on a barrier that nothing completes: the bounded wait runs out, records its site and
// the kernel returns normally (see bro_selftest_expire_wait).
__global__ void expire_wait_kernel(uint64_t budget_ns) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = bro::smem_u32(&bar);
  if (threadIdx.x == 0) {
    bro::mbar_init(b, 1);
    bro::mbar_fence_init();
  }
  __syncwarp();
  bro::mbar_wait(b, 0u, bro::SITE_SELF_TEST, budget_ns);
}

// h = bf16(silu(gate) * up), 8 values per thread (the producer alone; see rqd::silu_mul).
__global__ void __launch_bounds__(256) swiglu_kernel(const uint16_t* gate, const uint16_t* up, int64_t M, int64_t K,
                                                     int64_t ldg, int64_t ldu, uint16_t* h, int64_t ldh) {
  bro::griddep_wait();
  bro::griddep_launch_dependents();
  const int64_t chunks = K >> 3, total = M * chunks;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / chunks, c = i - row * chunks;
    const uint4 g = __ldg(reinterpret_cast<const uint4*>(gate + row * ldg + c * 8));
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(up + row * ldu + c * 8));
    *reinterpret_cast<uint4*>(h + row * ldh + c * 8) = bro::rqd::swiglu_bf16x8(g, u);
  }
}

// ---- rotate + quantise ---------------------------------------------------------------------------
bro_status launch_rotate_quantize(const void* x, int64_t M, int64_t K, int64_t ldx, int block,
                                  const void* signs, void* codes, void* scales, bro_layout layout,
                                  uint32_t flags, cudaStream_t st, const void* up = nullptr, int64_t ldu = 0) {
  // (up != nullptr: x is the gate of the fused producer, the rotated tensor is silu(x) * up)
  if (up && (ldu < K || ldu % 8 != 0)) return ldu < K ? BRO_ERR_SHAPE : BRO_ERR_ALIGN;
  if (up && !aligned(up, 16)) return BRO_ERR_ALIGN;
  if (up && block == 0) return BRO_ERR_UNSUPPORTED;
  if (M < 0 || K <= 0 || K % kGroup != 0 || ldx < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (M == 0 && (layout == BRO_LAYOUT_CANONICAL || layout == BRO_LAYOUT_GEMM)) return BRO_OK;
  if (!x || !codes || !scales) return BRO_ERR_NULL;
  if (layout != BRO_LAYOUT_CANONICAL && layout != BRO_LAYOUT_GEMM) return BRO_ERR_SHAPE;
  const int64_t B = block == 0 ? K : block;
  // 32, 64, 128 or K; also 2, 4, 8, 16 — a rotation inside the MX group (Sec. 5.2 sweeps the dimension both ways)
  if (block != 0 && !(block >= 2 && block <= 128 && is_pow2(block))) return BRO_ERR_SHAPE;
  if (K % B != 0) return BRO_ERR_SHAPE;
  if (block == 0 && (!is_pow2(K) || K < 32 || K > 32768)) return BRO_ERR_UNSUPPORTED;
  if (ldx % 8 != 0 || !aligned(x, 16) || !aligned(codes, 16) || !aligned(scales, 16) || !aligned(signs, 16))
    return BRO_ERR_ALIGN;
  if (M == 0) return BRO_OK;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;

  if (B > 128) {
    return bro::rqg::launch(x, M, K, ldx, signs, codes, scales, nullptr, 0, layout, gemm_scale_kblocks(K), di.sm_count, st);
  }

  // Register-streaming kernel by default (the TMA-ring kernel when the task index would not fit
  // 31 bits): it wins for block 32 at every size and for small inputs; for blocks of 64 / 128 on
  // large inputs its extra registers cost occupancy and the TMA ring is faster.  The flags of the
  // *_ex entry point override the choice.
  const bool can_direct = bro::rqd::supports(M, K, layout, gemm_scale_kblocks(K));
  bool direct = can_direct && (B <= 32 || M * K <= ((int64_t)1 << 23));
  if (flags & BRO_FLAG_RQ_TMA_RING) direct = false;
  else if (flags & BRO_FLAG_RQ_DIRECT) direct = can_direct;
  if (B < 32) {                   // blocks below the MX group exist in the register-streaming kernel only
    if (!can_direct) return BRO_ERR_UNSUPPORTED;
    direct = true;
  }
  if (up) {                       // the fused producer exists in the register-streaming kernel only
    if (!can_direct) return BRO_ERR_UNSUPPORTED;
    direct = true;
  }
  if (direct)
    return bro::rqd::launch(x, M, K, ldx, log2_of(B), signs, codes, scales, layout,
                            gemm_scale_kblocks(K), di.sm_count, st, up, ldu);

  CUtensorMap tmx;
  rc = make_map_2d(&tmx, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, x, (uint64_t)K, (uint64_t)M,
                   (uint64_t)ldx * 2, bro::rq::kBoxCols, bro::rq::kTileRows, CU_TENSOR_MAP_SWIZZLE_128B);
  if (rc != BRO_OK) return rc;

  Params p;
  p.M = M;
  p.K = K;
  p.tiles_m = ceil_div(M, bro::rq::kTileRows);
  p.tiles_k = layout == BRO_LAYOUT_GEMM ? gemm_scale_kblocks(K) : ceil_div(K, bro::rq::kTileCols);
  p.codes = static_cast<uint8_t*>(codes);
  p.scales = static_cast<uint8_t*>(scales);
  p.scale_kblocks = gemm_scale_kblocks(K);
  p.layout = (int)layout;
  p.signs = static_cast<const uint16_t*>(signs);
  const int64_t tiles = p.tiles_m * p.tiles_k;
  const int grid = (int)(tiles < di.sm_count ? tiles : di.sm_count);

  // (All six instantiations share one function-pointer type, so the opt-in to large dynamic
  // shared memory is kept per instantiation, per device.)
  auto go = [&](void (*kernel)(CUtensorMap, Params), int which) -> bro_status {
    static bro::DeviceOnce once[6];
    bro_status r = bro::device_once(once[which], nullptr, [&](int*) { return set_smem(kernel, bro::rq::kSmemBytes); });
    if (r != BRO_OK) return r;
    return bro::cuda_ok(bro::launch_kernel(kernel, (unsigned)grid, bro::rq::kThreads, bro::rq::kSmemBytes, st, 1, tmx, p),
                        "rotate_quantize launch")
               ? BRO_OK
               : BRO_ERR_CUDA;
  };
  if (signs) {
    switch (B) {
      case 32: return go(bro::rq::rotate_quantize_kernel<5, true>, 3);
      case 64: return go(bro::rq::rotate_quantize_kernel<6, true>, 4);
      default: return go(bro::rq::rotate_quantize_kernel<7, true>, 5);
    }
  }
  switch (B) {
    case 32: return go(bro::rq::rotate_quantize_kernel<5, false>, 0);
    case 64: return go(bro::rq::rotate_quantize_kernel<6, false>, 1);
    default: return go(bro::rq::rotate_quantize_kernel<7, false>, 2);
  }
}

}  // namespace

// =================================================================================================
extern "C" {

const char* bro_last_cuda_error(void) { return bro::g_last_cuda_error; }

const char* bro_status_string(bro_status s) {
  switch (s) {
    case BRO_OK: return "BRO_OK";
    case BRO_ERR_NULL: return "BRO_ERR_NULL";
    case BRO_ERR_SHAPE: return "BRO_ERR_SHAPE";
    case BRO_ERR_ALIGN: return "BRO_ERR_ALIGN";
    case BRO_ERR_UNSUPPORTED: return "BRO_ERR_UNSUPPORTED";
    case BRO_ERR_WORKSPACE: return "BRO_ERR_WORKSPACE";
    case BRO_ERR_CUDA: return "BRO_ERR_CUDA";
    case BRO_ERR_TIMEOUT: return "BRO_ERR_TIMEOUT";
    case BRO_ERR_ARCH: return "BRO_ERR_ARCH";
  }
  return "BRO_ERR_UNKNOWN";
}

size_t bro_codes_bytes(int64_t rows, int64_t K) {
  if (rows < 0 || K <= 0 || K % kGroup != 0) return 0;
  return (size_t)rows * (size_t)(K / 2);
}

size_t bro_scales_bytes(int64_t rows, int64_t K, bro_layout layout) {
  if (rows < 0 || K <= 0 || K % kGroup != 0) return 0;
  if (layout == BRO_LAYOUT_CANONICAL) return (size_t)rows * (size_t)(K / kGroup);
  if (layout == BRO_LAYOUT_GEMM) return (size_t)ceil_div(rows, 128) * (size_t)gemm_scale_kblocks(K) * 512;
  return 0;
}

size_t bro_scale_offset(int64_t row, int64_t group, int64_t rows, int64_t K, bro_layout layout) {
  (void)rows;
  if (layout == BRO_LAYOUT_CANONICAL) return (size_t)(row * (K / kGroup) + group);
  return (size_t)(((row / 128) * gemm_scale_kblocks(K) + group / 4) * 512 + (row % 32) * 16 +
                  ((row % 128) / 32) * 4 + (group % 4));
}

size_t bro_gemm_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  return bro::gemm::workspace_bytes(M, N, K);
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t bro_linear_workspace_bytes(int64_t M, int64_t N, int64_t K) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0) return 0;
  return align_up(bro_codes_bytes(M, K), 1024) + align_up(bro_scales_bytes(M, K, BRO_LAYOUT_GEMM), 1024) +
         align_up(bro_gemm_workspace_bytes(M, N, K), 1024);
}

bro_status bro_last_device_status_ex(void* stream, int* site) {
  if (site) *site = 0;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!bro::cuda_ok(cudaStreamSynchronize(st), "cudaStreamSynchronize")) return BRO_ERR_CUDA;
  unsigned int v = 0, zero = 0;
  if (!bro::cuda_ok(cudaMemcpyFromSymbol(&v, bro::g_device_status, sizeof(v)), "read of the device status word"))
    return BRO_ERR_CUDA;
  if (v != 0 && !bro::cuda_ok(cudaMemcpyToSymbol(bro::g_device_status, &zero, sizeof(zero)), "reset of the device status word"))
    return BRO_ERR_CUDA;
  if (site) *site = (int)(v >> 8);
  return (bro_status)(v & 0xFF);
}

bro_status bro_last_device_status(void* stream) { return bro_last_device_status_ex(stream, nullptr); }

bro_status bro_selftest_expire_wait(uint64_t budget_ns, void* stream) {
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  if (budget_ns < 1000ull) budget_ns = 1000ull;
  if (budget_ns > 100ull * 1000ull * 1000ull) budget_ns = 100ull * 1000ull * 1000ull;
  expire_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(budget_ns);
  return bro::cuda_ok(cudaGetLastError(), "self-test launch") ? BRO_OK : BRO_ERR_CUDA;
}

bro_status bro_rotate_quantize_mxfp4(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                     void* codes, void* scales, bro_layout layout, void* stream) {
  return launch_rotate_quantize(x_bf16, M, K, ldx, block, nullptr, codes, scales, layout, 0u,
                                static_cast<cudaStream_t>(stream));
}

bro_status bro_rotate_quantize_mxfp4_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                        const void* signs_bf16, void* codes, void* scales, bro_layout layout,
                                        uint32_t flags, void* stream) {
  return launch_rotate_quantize(x_bf16, M, K, ldx, block, signs_bf16, codes, scales, layout, flags,
                                static_cast<cudaStream_t>(stream));
}

bro_status bro_rotate_quantize_mxfp4_rs(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                        const void* signs_bf16, void* codes, void* scales, bro_layout layout,
                                        void* stream) {
  return launch_rotate_quantize(x_bf16, M, K, ldx, block, signs_bf16, codes, scales, layout, 0u,
                                static_cast<cudaStream_t>(stream));
}

// Rotation sizes of the analysis calls: 0 (= K), 1 (none), and the powers of two from 2 to 128 — below,
// at and above the MX group (Sec. 5.2 sweeps the rotation dimension both ways).
static bool analysis_block(int block) {
  return block == 0 || (block >= 1 && block <= 128 && (block & (block - 1)) == 0);
}

bro_status bro_group_quant_error_fmt(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                     const void* signs_bf16, bro_format format, float* mse, void* stream) {
  if ((int)format < 0 || (int)format > 3) return BRO_ERR_SHAPE;
  if (M < 0 || K <= 0 || K % kGroup != 0 || ldx < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (M == 0) return BRO_OK;
  if (!x_bf16 || !mse) return BRO_ERR_NULL;
  const int64_t B = block == 0 ? K : block;
  if (!analysis_block(block)) return BRO_ERR_SHAPE;
  if (K % B != 0) return BRO_ERR_SHAPE;
  if (block == 0 && (!is_pow2(K) || K < 32 || K > 32768)) return BRO_ERR_UNSUPPORTED;
  if (ldx % 8 != 0 || !aligned(x_bf16, 16) || !aligned(mse, 4) || !aligned(signs_bf16, 16)) return BRO_ERR_ALIGN;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (B < 32)   // no rotation, or one inside the MX group
    return bro::fq::launch(x_bf16, M, K, ldx, (int)B, signs_bf16, (int)format, nullptr, 0, mse, nullptr, di.sm_count, st);
  if (B > 128)
    return bro::rqg::launch(x_bf16, M, K, ldx, signs_bf16, nullptr, nullptr, mse, (int)format, BRO_LAYOUT_CANONICAL, 0, di.sm_count, st);
  if (!bro::rqd::supports(M, K, BRO_LAYOUT_CANONICAL, 0)) return BRO_ERR_UNSUPPORTED;
  return bro::rqd::launch_stats(x_bf16, M, K, ldx, B == 32 ? 5 : (B == 64 ? 6 : 7), signs_bf16, (int)format, mse, nullptr, di.sm_count, st);
}

// ---- simulated quantisation ----------------------------------------------------------------------
size_t bro_fake_quantize_workspace_bytes(int64_t M, bro_format format) {
  const bool rows = format == BRO_FMT_INT4_ROW_SYM || format == BRO_FMT_INT4_ROW_ASYM;
  return (rows && M > 0) ? (size_t)M * 8 : 0;
}

bro_status bro_rotate_fake_quantize_ws(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                       const void* signs_bf16, bro_format format, float* deq, int64_t ldd,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  if ((int)format < 0 || (int)format > (int)BRO_FMT_NONE) return BRO_ERR_SHAPE;
  if (M < 0 || K <= 0 || K % kGroup != 0 || ldx < K || ldd < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (!analysis_block(block)) return BRO_ERR_SHAPE;
  const int64_t B = block == 0 ? K : block;
  if (K % B != 0) return BRO_ERR_SHAPE;
  if (block == 0 && (!is_pow2(K) || K < 32 || K > 32768)) return BRO_ERR_UNSUPPORTED;
  if (M == 0) return BRO_OK;
  if (!x_bf16 || !deq) return BRO_ERR_NULL;
  if (ldx % 8 != 0 || ldd % 4 != 0 || !aligned(x_bf16, 16) || !aligned(deq, 16) || !aligned(signs_bf16, 16))
    return BRO_ERR_ALIGN;
  const size_t need = bro_fake_quantize_workspace_bytes(M, format);
  if (need > 0 && (!workspace || workspace_bytes < need)) return BRO_ERR_WORKSPACE;
  if (need > 0 && !aligned(workspace, 8)) return BRO_ERR_ALIGN;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint32_t* rowstats = need > 0 ? static_cast<uint32_t*>(workspace) : nullptr;
  if (rowstats) {
    // per-row formats: a first pass leaves every row's range in the workspace
    if (!bro::cuda_ok(cudaMemsetAsync(rowstats, 0, need, st), "cudaMemsetAsync(row ranges)")) return BRO_ERR_CUDA;
    rc = B > 128 ? bro::rqg::launch(x_bf16, M, K, ldx, signs_bf16, nullptr, nullptr, nullptr, (int)format, BRO_LAYOUT_CANONICAL,
                                    0, di.sm_count, st, nullptr, 0, rowstats, true)
                 : bro::fq::launch(x_bf16, M, K, ldx, (int)B, signs_bf16, (int)format, nullptr, 0, nullptr, nullptr,
                                   di.sm_count, st, rowstats);
    if (rc != BRO_OK) return rc;
  }
  if (B > 128)
    return bro::rqg::launch(x_bf16, M, K, ldx, signs_bf16, nullptr, nullptr, nullptr, (int)format, BRO_LAYOUT_CANONICAL, 0,
                            di.sm_count, st, deq, ldd, rowstats, false);
  return bro::fq::launch(x_bf16, M, K, ldx, (int)B, signs_bf16, (int)format, deq, ldd, nullptr, nullptr, di.sm_count, st,
                         rowstats);
}

bro_status bro_rotate_fake_quantize(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                    const void* signs_bf16, bro_format format, float* deq, int64_t ldd,
                                    void* stream) {
  return bro_rotate_fake_quantize_ws(x_bf16, M, K, ldx, block, signs_bf16, format, deq, ldd, nullptr, 0, stream);
}

// ---- scale statistics ----------------------------------------------------------------------------
bro_status bro_group_scale_bytes(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                 const void* signs_bf16, uint8_t* scales, void* stream) {
  if (M < 0 || K <= 0 || K % kGroup != 0 || ldx < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (!analysis_block(block)) return BRO_ERR_SHAPE;
  const int64_t B = block == 0 ? K : block;
  if (K % B != 0) return BRO_ERR_SHAPE;
  if (block == 0 && (!is_pow2(K) || K < 32 || K > 32768)) return BRO_ERR_UNSUPPORTED;
  if (M == 0) return BRO_OK;
  if (!x_bf16 || !scales) return BRO_ERR_NULL;
  if (ldx % 8 != 0 || !aligned(x_bf16, 16) || !aligned(signs_bf16, 16)) return BRO_ERR_ALIGN;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (block == 1) {
    // the identity rotation: a sign flip does not change a magnitude, so the signs play no part
    const unsigned grid = bro::stats::grid_for(M * (K / 32), 256, di.sm_count, 8);
    return bro::cuda_ok(bro::launch_kernel(bro::stats::group_scale_bytes_identity, grid, 256, 0, st, 1,
                                           static_cast<const uint16_t*>(x_bf16), M, K, ldx, scales),
                        "group_scale_bytes launch")
               ? BRO_OK
               : BRO_ERR_CUDA;
  }
  if (B < 32)   // a rotation inside the MX group
    return bro::fq::launch(x_bf16, M, K, ldx, (int)B, signs_bf16, 0, nullptr, 0, nullptr, scales, di.sm_count, st);
  if (B > 128)
    return bro::rqg::launch(x_bf16, M, K, ldx, signs_bf16, nullptr, scales, nullptr, bro::rq::kFormatScaleOnly,
                            BRO_LAYOUT_CANONICAL, 0, di.sm_count, st);
  if (!bro::rqd::supports(M, K, BRO_LAYOUT_CANONICAL, 0)) return BRO_ERR_UNSUPPORTED;
  return bro::rqd::launch_stats(x_bf16, M, K, ldx, B == 32 ? 5 : (B == 64 ? 6 : 7), signs_bf16,
                                bro::rq::kFormatScaleOnly, nullptr, scales, di.sm_count, st);
}

size_t bro_outlier_workspace_bytes(void) { return bro::stats::kWorkspaceBytes; }

bro_status bro_outlier_groups(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int64_t top_ppm,
                              uint8_t* mask, uint32_t* info, void* workspace, size_t workspace_bytes,
                              void* stream) {
  if (M < 0 || K <= 0 || K % kGroup != 0 || ldx < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (top_ppm <= 0 || top_ppm > 1000000) return BRO_ERR_SHAPE;
  if (M == 0) return BRO_OK;
  if (!x_bf16 || !mask || !info || !workspace) return BRO_ERR_NULL;
  if (ldx % 8 != 0 || !aligned(x_bf16, 16) || !aligned(info, 16) || !aligned(workspace, 16)) return BRO_ERR_ALIGN;
  if (workspace_bytes < bro::stats::kWorkspaceBytes) return BRO_ERR_WORKSPACE;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned long long* hist = static_cast<unsigned long long*>(workspace);
  if (!bro::cuda_ok(cudaMemsetAsync(hist, 0, (size_t)bro::stats::kMagBins * 8, st), "cudaMemsetAsync(histogram)"))
    return BRO_ERR_CUDA;
  static bro::DeviceOnce once;
  const int smem = bro::stats::kMagBins * 4;
  rc = bro::device_once(once, nullptr, [&](int*) { return set_smem(bro::stats::magnitude_histogram, smem); });
  if (rc != BRO_OK) return rc;
  const uint16_t* x = static_cast<const uint16_t*>(x_bf16);
  const unsigned hgrid = bro::stats::grid_for(M * (K / 8), 512, di.sm_count, 1);
  if (!bro::cuda_ok(bro::launch_kernel(bro::stats::magnitude_histogram, hgrid, 512, (size_t)smem, st, 1, x, M, K, ldx, hist),
                    "magnitude_histogram launch"))
    return BRO_ERR_CUDA;
  const unsigned long long n = (unsigned long long)M * (unsigned long long)K;
  unsigned long long k = (n * (unsigned long long)top_ppm + 999999ull) / 1000000ull;
  if (k < 1) k = 1;
  if (!bro::cuda_ok(bro::launch_kernel(bro::stats::find_threshold, 1u, 1024u, 0, st, 1,
                                       static_cast<const unsigned long long*>(hist), k, info),
                    "find_threshold launch"))
    return BRO_ERR_CUDA;
  const unsigned mgrid = bro::stats::grid_for(M * (K / 32), 256, di.sm_count, 8);
  return bro::cuda_ok(bro::launch_kernel(bro::stats::outlier_group_mask, mgrid, 256, 0, st, 1, x, M, K, ldx,
                                         static_cast<const uint32_t*>(info), mask),
                      "outlier_group_mask launch")
             ? BRO_OK
             : BRO_ERR_CUDA;
}

bro_status bro_scale_histogram(const uint8_t* scales, const uint8_t* mask, int64_t n_groups, uint64_t* hist,
                               void* stream) {
  if (n_groups < 0) return BRO_ERR_SHAPE;
  if (!hist) return BRO_ERR_NULL;
  if (!aligned(hist, 8)) return BRO_ERR_ALIGN;
  if (n_groups > 0 && (!scales || !mask)) return BRO_ERR_NULL;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!bro::cuda_ok(cudaMemsetAsync(hist, 0, 2 * 256 * sizeof(uint64_t), st), "cudaMemsetAsync(scale histogram)"))
    return BRO_ERR_CUDA;
  if (n_groups == 0) return BRO_OK;
  const unsigned grid = bro::stats::grid_for(n_groups, 256 * 16, di.sm_count, 4);
  return bro::cuda_ok(bro::launch_kernel(bro::stats::scale_histogram, grid, 256, 0, st, 1, scales, mask, n_groups,
                                         reinterpret_cast<unsigned long long*>(hist)),
                      "scale_histogram launch")
             ? BRO_OK
             : BRO_ERR_CUDA;
}

bro_status bro_scale_inflation(const uint8_t* scales_before, const uint8_t* scales_after, const uint8_t* mask,
                               int64_t n_groups, uint64_t* counts, void* stream) {
  if (n_groups < 0) return BRO_ERR_SHAPE;
  if (!counts) return BRO_ERR_NULL;
  if (!aligned(counts, 8)) return BRO_ERR_ALIGN;
  if (n_groups > 0 && (!scales_before || !scales_after || !mask)) return BRO_ERR_NULL;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (!bro::cuda_ok(cudaMemsetAsync(counts, 0, 6 * sizeof(uint64_t), st), "cudaMemsetAsync(inflation counts)"))
    return BRO_ERR_CUDA;
  if (n_groups == 0) return BRO_OK;
  const unsigned grid = bro::stats::grid_for(n_groups, 256 * 16, di.sm_count, 4);
  return bro::cuda_ok(bro::launch_kernel(bro::stats::scale_inflation, grid, 256, 0, st, 1, scales_before, scales_after, mask,
                                         n_groups, reinterpret_cast<unsigned long long*>(counts)),
                      "scale_inflation launch")
             ? BRO_OK
             : BRO_ERR_CUDA;
}

bro_status bro_group_quant_error(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                                 const void* signs_bf16, float* mse, void* stream) {
  return bro_group_quant_error_fmt(x_bf16, M, K, ldx, block, signs_bf16, BRO_FMT_MXFP4, mse, stream);
}

bro_status bro_pack_weights_rs(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                               const void* signs_bf16, void* wcodes, void* wscales, void* stream) {
  return launch_rotate_quantize(w_bf16, N, K, ldw, block, signs_bf16, wcodes, wscales, BRO_LAYOUT_GEMM, 0u,
                                static_cast<cudaStream_t>(stream));
}

bro_status bro_pack_weights(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                            void* wcodes, void* wscales, void* stream) {
  return launch_rotate_quantize(w_bf16, N, K, ldw, block, nullptr, wcodes, wscales, BRO_LAYOUT_GEMM, 0u,
                                static_cast<cudaStream_t>(stream));
}

static bro_status gemm_impl(const void* acodes, const void* ascales, const void* wcodes, const void* wscales,
                            int64_t M, int64_t N, int64_t K, void* y, int64_t ldy, bro_out_dtype out_dtype,
                            void* workspace, size_t workspace_bytes, uint32_t flags, void* stream, bool w_static) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0 || ldy < N) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || N > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (out_dtype != BRO_OUT_BF16 && out_dtype != BRO_OUT_F32) return BRO_ERR_SHAPE;
  if (M == 0 || N == 0) return BRO_OK;
  if (!acodes || !ascales || !wcodes || !wscales || !y) return BRO_ERR_NULL;
  const int64_t esz = out_dtype == BRO_OUT_BF16 ? 2 : 4;
  if (!aligned(acodes, 128) || !aligned(wcodes, 128) || !aligned(ascales, 128) || !aligned(wscales, 128) ||
      !aligned(y, 16) || (ldy * esz) % 16 != 0)
    return BRO_ERR_ALIGN;
  const size_t need = bro_gemm_workspace_bytes(M, N, K);
  if (need > 0 && (!workspace || workspace_bytes < need)) return BRO_ERR_WORKSPACE;
  if (M == 0 || N == 0) return BRO_OK;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  // Two kernels.  The two-CTA kernel (256 x 256 tiles, cta_group::2) moves a third fewer bytes into
  // shared memory per flop and measures 3-7 % faster once a problem has at least two rounds of
  // 256 x 256 tiles and tiles long enough (K >= 4096) to amortise its costlier tile hand-over; below
  // that the single-CTA kernel wins (half-width units for the last round, 128-row granularity, cheaper
  // prologue).  The flags of the *_ex entry point force either.
  bool pair = (flags & BRO_FLAG_GEMM_PAIR) != 0;
  if (!(flags & (BRO_FLAG_GEMM_PAIR | BRO_FLAG_GEMM_SINGLE | BRO_FLAG_GEMM_TILE_N128 | BRO_FLAG_GEMM_TILE_N256)))
    pair = K >= 4096 && ceil_div(M, 256) * ceil_div(N, 256) >= 2 * (int64_t)(di.sm_count / 2);
  if (pair)
    return bro::gemm2::launch(acodes, ascales, wcodes, wscales, M, N, K, y, ldy, (int)out_dtype, flags, di.sm_count,
                              static_cast<cudaStream_t>(stream));
  return bro::gemm::launch(acodes, ascales, wcodes, wscales, M, N, K, y, ldy, (int)out_dtype, workspace,
                           workspace_bytes, flags, di.sm_count, static_cast<cudaStream_t>(stream), w_static);
}

bro_status bro_gemm_mxfp4(const void* acodes, const void* ascales, const void* wcodes,
                          const void* wscales, int64_t M, int64_t N, int64_t K, void* y, int64_t ldy,
                          bro_out_dtype out_dtype, void* workspace, size_t workspace_bytes,
                          void* stream) {
  // the weights may have been written by the kernel just before this one: no early fetch
  return gemm_impl(acodes, ascales, wcodes, wscales, M, N, K, y, ldy, out_dtype, workspace, workspace_bytes, 0u,
                   stream, false);
}

bro_status bro_gemm_mxfp4_ex(const void* acodes, const void* ascales, const void* wcodes, const void* wscales,
                             int64_t M, int64_t N, int64_t K, void* y, int64_t ldy, bro_out_dtype out_dtype,
                             void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  return gemm_impl(acodes, ascales, wcodes, wscales, M, N, K, y, ldy, out_dtype, workspace, workspace_bytes, flags,
                   stream, false);
}

static bro_status linear_impl(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block, const void* signs,
                              const void* wcodes, const void* wscales, int64_t N, void* y_bf16, int64_t ldy,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0) return BRO_ERR_SHAPE;
  if (M == 0 || N == 0) return BRO_OK;
  if (!x_bf16 || !wcodes || !wscales || !y_bf16 || !workspace) return BRO_ERR_NULL;
  if (!aligned(workspace, 1024)) return BRO_ERR_ALIGN;
  if (workspace_bytes < bro_linear_workspace_bytes(M, N, K)) return BRO_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* acodes = ws;
  uint8_t* ascales = acodes + align_up(bro_codes_bytes(M, K), 1024);
  uint8_t* gws = ascales + align_up(bro_scales_bytes(M, K, BRO_LAYOUT_GEMM), 1024);
  bro_status rc = launch_rotate_quantize(x_bf16, M, K, ldx, block, signs, acodes, ascales, BRO_LAYOUT_GEMM, flags,
                                         static_cast<cudaStream_t>(stream));
  if (rc != BRO_OK) return rc;
  // The packed weights are older than the rotate+quantize kernel just enqueued, which signals its
  // dependents only after its own wait: the GEMM may fetch its first weight tiles early.
  return gemm_impl(acodes, ascales, wcodes, wscales, M, N, K, y_bf16, ldy, BRO_OUT_BF16, gws,
                   bro_gemm_workspace_bytes(M, N, K), flags, stream, true);
}

bro_status bro_linear(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block, const void* wcodes,
                      const void* wscales, int64_t N, void* y_bf16, int64_t ldy, void* workspace,
                      size_t workspace_bytes, void* stream) {
  return linear_impl(x_bf16, M, K, ldx, block, nullptr, wcodes, wscales, N, y_bf16, ldy, workspace,
                     workspace_bytes, 0u, stream);
}

bro_status bro_linear_ex(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block, const void* signs_bf16,
                         const void* wcodes, const void* wscales, int64_t N, void* y_bf16, int64_t ldy,
                         void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
  return linear_impl(x_bf16, M, K, ldx, block, signs_bf16, wcodes, wscales, N, y_bf16, ldy, workspace,
                     workspace_bytes, flags, stream);
}

bro_status bro_linear_rs(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block, const void* signs_bf16,
                         const void* wcodes, const void* wscales, int64_t N, void* y_bf16, int64_t ldy,
                         void* workspace, size_t workspace_bytes, void* stream) {
  if (!signs_bf16) return BRO_ERR_NULL;
  return linear_impl(x_bf16, M, K, ldx, block, signs_bf16, wcodes, wscales, N, y_bf16, ldy, workspace,
                     workspace_bytes, 0u, stream);
}

bro_status bro_swiglu_rotate_quantize_mxfp4(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K, int64_t ldg,
                                            int64_t ldu, int block, const void* signs_bf16, void* codes, void* scales,
                                            bro_layout layout, void* stream) {
  if (M > 0 && !up_bf16) return BRO_ERR_NULL;
  if (block == 0) return BRO_ERR_UNSUPPORTED;
  return launch_rotate_quantize(gate_bf16, M, K, ldg, block, signs_bf16, codes, scales, layout, 0u,
                                static_cast<cudaStream_t>(stream), up_bf16, ldu);
}

bro_status bro_swiglu_bf16(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K, int64_t ldg, int64_t ldu,
                           void* h_bf16, int64_t ldh, void* stream) {
  if (M < 0 || K <= 0 || K % 8 != 0 || ldg < K || ldu < K || ldh < K) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (M == 0) return BRO_OK;
  if (!gate_bf16 || !up_bf16 || !h_bf16) return BRO_ERR_NULL;
  if (ldg % 8 != 0 || ldu % 8 != 0 || ldh % 8 != 0 || !aligned(gate_bf16, 16) || !aligned(up_bf16, 16) || !aligned(h_bf16, 16))
    return BRO_ERR_ALIGN;
  DeviceInfo di;
  bro_status rc = device_info(&di);
  if (rc != BRO_OK) return rc;
  const int64_t want = (M * (K / 8) + 255) / 256, cap = (int64_t)di.sm_count * 8;
  return bro::cuda_ok(bro::launch_kernel(swiglu_kernel, (unsigned)(want < cap ? want : cap), 256, 0,
                                         static_cast<cudaStream_t>(stream), 1, static_cast<const uint16_t*>(gate_bf16),
                                         static_cast<const uint16_t*>(up_bf16), M, K, ldg, ldu,
                                         static_cast<uint16_t*>(h_bf16), ldh),
                      "swiglu launch")
             ? BRO_OK
             : BRO_ERR_CUDA;
}

bro_status bro_swiglu_linear(const void* gate_bf16, const void* up_bf16, int64_t M, int64_t K, int64_t ldg, int64_t ldu,
                             int block, const void* signs_bf16, const void* wcodes, const void* wscales, int64_t N,
                             void* y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes, void* stream) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0) return BRO_ERR_SHAPE;
  if (M == 0 || N == 0) return BRO_OK;
  if (!gate_bf16 || !up_bf16 || !wcodes || !wscales || !y_bf16 || !workspace) return BRO_ERR_NULL;
  if (block == 0) return BRO_ERR_UNSUPPORTED;
  if (!aligned(workspace, 1024)) return BRO_ERR_ALIGN;
  if (workspace_bytes < bro_linear_workspace_bytes(M, N, K)) return BRO_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint8_t* acodes = ws;
  uint8_t* ascales = acodes + align_up(bro_codes_bytes(M, K), 1024);
  uint8_t* gws = ascales + align_up(bro_scales_bytes(M, K, BRO_LAYOUT_GEMM), 1024);
  bro_status rc = launch_rotate_quantize(gate_bf16, M, K, ldg, block, signs_bf16, acodes, ascales, BRO_LAYOUT_GEMM, 0u,
                                         static_cast<cudaStream_t>(stream), up_bf16, ldu);
  if (rc != BRO_OK) return rc;
  return gemm_impl(acodes, ascales, wcodes, wscales, M, N, K, y_bf16, ldy, BRO_OUT_BF16, gws,
                   bro_gemm_workspace_bytes(M, N, K), 0u, stream, true);
}

bro_status bro_pack_weights_desc(const void* w_bf16, int64_t N, int64_t K, int64_t ldw, int block,
                                 const void* signs_bf16, void* wcodes, void* wscales, bro_packed_weights* desc,
                                 void* stream) {
  if (!desc) return BRO_ERR_NULL;
  desc->magic = 0;          // stays invalid unless the packing was enqueued
  const bro_status rc = launch_rotate_quantize(w_bf16, N, K, ldw, block, signs_bf16, wcodes, wscales, BRO_LAYOUT_GEMM, 0u,
                                               static_cast<cudaStream_t>(stream));
  if (rc != BRO_OK) return rc;
  desc->magic = BRO_WEIGHTS_MAGIC;
  desc->version = BRO_WEIGHTS_VERSION;
  desc->N = N;
  desc->K = K;
  desc->block = block;
  desc->randomised = signs_bf16 ? 1 : 0;
  desc->codes = wcodes;
  desc->scales = wscales;
  return BRO_OK;
}

bro_status bro_linear_packed(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block, const void* signs_bf16,
                             const bro_packed_weights* weights, void* y_bf16, int64_t ldy, void* workspace,
                             size_t workspace_bytes, void* stream) {
  if (!weights) return BRO_ERR_NULL;
  if (weights->magic != BRO_WEIGHTS_MAGIC || weights->version != BRO_WEIGHTS_VERSION) return BRO_ERR_UNSUPPORTED;
  // the rotation only cancels, (x R)(W R)^T = x W^T, when both sides used the same R
  if (weights->K != K || weights->block != block || (weights->randomised != 0) != (signs_bf16 != nullptr))
    return BRO_ERR_SHAPE;
  return linear_impl(x_bf16, M, K, ldx, block, signs_bf16, weights->codes, weights->scales, weights->N, y_bf16, ldy,
                     workspace, workspace_bytes, 0u, stream);
}

bro_status bro_linear_host(const void* x_host_bf16, int64_t M, int64_t K, int block, const void* wcodes,
                           const void* wscales, int64_t N, void* y_host_bf16, void* x_stage, void* y_stage,
                           void* workspace, size_t workspace_bytes, void* stream) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0) return BRO_ERR_SHAPE;
  if (M == 0 || N == 0) return BRO_OK;
  if (!x_host_bf16 || !y_host_bf16 || !x_stage || !y_stage) return BRO_ERR_NULL;
  if (N % 8 != 0) return BRO_ERR_SHAPE;   // dense y staging needs a 16-byte row pitch
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(x_stage, x_host_bf16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return BRO_ERR_CUDA;
  bro_status rc = bro_linear(x_stage, M, K, K, block, wcodes, wscales, N, y_stage, N, workspace,
                             workspace_bytes, stream);
  if (rc != BRO_OK) return rc;
  if (cudaMemcpyAsync(y_host_bf16, y_stage, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return BRO_ERR_CUDA;
  return BRO_OK;
}

// ---- bro_linear without a caller-provided workspace ---------------------------------------------
// The quantised activations (and any GEMM workspace) live in this array instead.  In host code the
// name is only a handle: the address a kernel can use comes from cudaGetSymbolAddress, looked up
// once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[BRO_STATIC_SCRATCH_BYTES];

bro_status bro_linear_static(const void* x_bf16, int64_t M, int64_t K, int64_t ldx, int block,
                             const void* wcodes, const void* wscales, int64_t N, void* y_bf16, int64_t ldy,
                             void* stream) {
  if (M < 0 || N < 0 || K <= 0 || K % kGroup != 0) return BRO_ERR_SHAPE;
  if (M > (int64_t)1 << 30 || N > (int64_t)1 << 30 || K > (int64_t)1 << 30) return BRO_ERR_SHAPE;
  if (M == 0 || N == 0) return BRO_OK;
  if (!x_bf16 || !wcodes || !wscales || !y_bf16) return BRO_ERR_NULL;
  const size_t codes_sz = align_up(bro_codes_bytes(M, K), 256);
  const size_t scales_sz = align_up(bro_scales_bytes(M, K, BRO_LAYOUT_GEMM), 256);
  const size_t gemm_sz = bro_gemm_workspace_bytes(M, N, K);
  const size_t need = codes_sz + scales_sz + gemm_sz;
  if (need > BRO_STATIC_SCRATCH_BYTES) {
    snprintf(bro::g_last_cuda_error, sizeof(bro::g_last_cuda_error),
             "bro_linear_static: this problem needs %zu bytes of scratch, the built-in array holds %zu; "
             "use bro_linear with a workspace", need, (size_t)BRO_STATIC_SCRATCH_BYTES);
    return BRO_ERR_WORKSPACE;
  }
  // Device address of the array, once per device, with that device current.
  static unsigned char* base_of[64] = {};
  static std::mutex mu;
  int dev = 0;
  if (!bro::cuda_ok(cudaGetDevice(&dev), "cudaGetDevice")) return BRO_ERR_CUDA;
  if (dev < 0 || dev >= 64) return BRO_ERR_UNSUPPORTED;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!base_of[dev]) {
      void* p = nullptr;
      if (!bro::cuda_ok(cudaGetSymbolAddress(&p, g_static_scratch), "cudaGetSymbolAddress(static scratch)") || !p)
        return BRO_ERR_CUDA;
      base_of[dev] = static_cast<unsigned char*>(p);
    }
    base = base_of[dev];
  }
  unsigned char* acodes = base;
  unsigned char* ascales = acodes + codes_sz;
  unsigned char* gws = ascales + scales_sz;
  bro_status rc = bro_rotate_quantize_mxfp4(x_bf16, M, K, ldx, block, acodes, ascales, BRO_LAYOUT_GEMM, stream);
  if (rc != BRO_OK) return rc;
  // (as in bro_linear: the packed weights are older than the kernel just enqueued, so the GEMM may
  // fetch its first weight tiles before that kernel has finished)
  return gemm_impl(acodes, ascales, wcodes, wscales, M, N, K, y_bf16, ldy, BRO_OUT_BF16, gemm_sz ? gws : nullptr,
                   gemm_sz, 0u, stream, true);
}

}  // extern "C"
