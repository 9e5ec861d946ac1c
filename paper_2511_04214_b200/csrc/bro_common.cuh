// Shared device-side helpers for libbro's sm_100a kernels: the device status word, bounded
// mbarrier waits, TMA (cp.async.bulk.tensor) wrappers and small PTX utilities.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <mutex>

#include "../../include/bro.h"

namespace bro {

// Host side: remember the text of the last failing CUDA call of this thread.
inline thread_local char g_last_cuda_error[256] = "";
inline bool cuda_ok(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return true;
  snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return false;
}

// One-time, per-device set-up of a kernel (shared-memory opt-in, occupancy query): host threads may
// race to the first launch, so the "done" table is guarded.  `init` returns BRO_OK and a positive
// value to remember; later calls on the same device get that value back without running it again.
struct DeviceOnce {
  std::mutex mu;
  int value[64] = {};
};
template <typename Init>
inline bro_status device_once(DeviceOnce& once, int* value_out, Init&& init) {
  int dev = 0;
  if (!cuda_ok(cudaGetDevice(&dev), "cudaGetDevice")) return BRO_ERR_CUDA;
  if (dev < 0 || dev >= 64) return BRO_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(once.mu);
  if (once.value[dev] == 0) {
    int v = 1;
    const bro_status rc = init(&v);
    if (rc != BRO_OK) return rc;
    once.value[dev] = v > 0 ? v : 1;
  }
  if (value_out) *value_out = once.value[dev];
  return BRO_OK;
}

// Launch with programmatic dependent launch enabled (and, if cluster_x > 1, that cluster width).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                 cudaStream_t st, unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid, 1, 1);
  cfg.blockDim = dim3(block, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[n].val.programmaticStreamSerializationAllowed = 1;
  ++n;
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// One status word per device (each device that loads the module gets its own instance).
// 0 = OK; otherwise (BRO_ERR_TIMEOUT) | (site << 8).  Kernels only ever move it away from 0.
__device__ unsigned int g_device_status = 0u;

// Time budget of one mbarrier wait, measured on the device's nanosecond timer (%globaltimer): a wait
// that has not completed after this long is declared lost.  No wait of a healthy run lasts longer than
// a kernel does (milliseconds); two seconds is far beyond that and still returns the GPU promptly.
constexpr uint64_t kWaitBudgetNs = 2000ull * 1000ull * 1000ull;

enum WaitSite : unsigned {
  SITE_RQ_FULL = 1, SITE_RQ_EMPTY = 2, SITE_RQ_DRAIN = 3,
  SITE_GEMM_FULL = 4, SITE_GEMM_EMPTY = 5, SITE_GEMM_ACC_FULL = 6, SITE_GEMM_ACC_EMPTY = 7,
  SITE_GEMM_DRAIN = 8, SITE_GEMM_TMEM = 9, SITE_SELF_TEST = 10
};

__device__ __forceinline__ void report_timeout(unsigned site) {
  atomicCAS(&g_device_status, 0u, (unsigned)BRO_ERR_TIMEOUT | (site << 8));
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier -------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false (after recording the site) if the phase has not completed within
// `budget_ns`.  The first probe costs nothing extra; the timer is read once per 32 failed probes
// (each failed try_wait already suspends the thread for a hardware-defined interval).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned site,
                                          uint64_t budget_ns = kWaitBudgetNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  do {
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try_wait(bar, parity)) return true;
  } while (global_timer_ns() - t0 <= budget_ns);
  report_timeout(site);
  return false;
}

// ---- TMA ------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled load global -> shared, completion counted in bytes on `bar`.  x is the innermost
// coordinate (elements of the map's data type); x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, int x, int y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// 3-D tiled load (x innermost; the same alignment rule for x).
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// 1-D bulk copy global -> shared (both addresses 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes,
                                             uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
      : "memory");
}

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the library is launched with the "programmatic stream serialization" attribute,
// so the next kernel in the stream may be scheduled while this one still runs: its CTAs start on
// SMs as they become free and run their prologue (barrier set-up, TMEM allocation, descriptor
// prefetch) early.  griddep_wait() blocks until all earlier grids in the stream have completed
// and their writes are visible; every thread calls it before its first access to global memory.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Forms for a converged warp in which one lane issues: `issue` is non-zero in that lane only.  The
// loop around them, and every address they take, stays warp-uniform.
__device__ __forceinline__ void mbar_arrive_expect_tx_if(uint32_t issue, uint32_t bar, uint32_t bytes) {
  asm volatile(
      "{ .reg .pred q; .reg .b64 st; setp.ne.b32 q, %2, 0;\n\t"
      "@q mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(bar),
      "r"(bytes), "r"(issue)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_if(uint32_t issue, uint32_t dst, const CUtensorMap* m, int x, int y,
                                               uint32_t bar) {
  asm volatile(
      "{ .reg .pred q; setp.ne.b32 q, %5, 0;\n\t"
      "@q cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3}], [%4]; }" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(bar), "r"(issue)
      : "memory");
}
__device__ __forceinline__ void bulk_load_1d_if(uint32_t issue, uint32_t dst, const void* src, uint32_t bytes,
                                                uint32_t bar) {
  asm volatile(
      "{ .reg .pred q; setp.ne.b32 q, %4, 0;\n\t"
      "@q cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3]; }" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar), "r"(issue)
      : "memory");
}
// Bounded wait executed by a whole converged warp; the result is the same in every lane.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, unsigned site) {
  const bool ok = mbar_wait(bar, parity, site);
  return __all_sync(0xFFFFFFFFu, ok);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "r"(addr));
  return v;
}

}  // namespace bro
