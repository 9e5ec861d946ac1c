// Analysis kernels: the scale statistics behind the paper's regular-block / outlier-block argument
// (Sec. 4.1: blocks without / with outliers; Sec. 4.2, Fig. 6 caption: outliers are the top 0.1 % of
// the activations by absolute value; App. A.3: under global rotation most regular blocks' scales grow,
// block rotation removes most of that growth).  All of it is integer work, so results are exact and
// independent of the order in which threads add their counts.
//
//   group_scale_bytes_identity   E8M0 byte of every group of 32 of the un-rotated input
//   magnitude_histogram          counts of the 32768 bf16 magnitude patterns (shared-memory histogram
//                                per CTA, merged with 64-bit atomics)
//   find_threshold               the k-th largest magnitude from that histogram (one CTA)
//   outlier_group_mask           groups holding a value at or above the threshold
//   scale_histogram              256-bin histograms of the scale bytes, regular and outlier groups
//   scale_inflation              per class: groups whose byte went down / stayed / went up
#pragma once

#include "bro_common.cuh"

namespace bro {
namespace stats {

constexpr int kMagBins = 32768;                       // bf16 magnitudes: the low 15 bits
constexpr size_t kWorkspaceBytes = (size_t)kMagBins * 8 + 64;

// max of the 15-bit magnitude patterns of 8 bf16 values (finite non-negative floats order like integers)
__device__ __forceinline__ uint32_t max_mag8(uint4 q) {
  uint32_t m = 0;
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m = max(m, w[i] & 0x7FFFu);
    m = max(m, (w[i] >> 16) & 0x7FFFu);
  }
  return m;
}

__device__ __forceinline__ uint32_t group_max_mag(const uint16_t* x, int64_t row, int64_t ldx, int64_t g) {
  const uint4* src = reinterpret_cast<const uint4*>(x + row * ldx + g * 32);
  uint32_t m = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) m = max(m, max_mag8(__ldg(src + j)));
  return m;
}

// One thread per group.  The byte is max(expfield(amax) - 2, 0) with expfield the 8-bit exponent of
// amax as fp32 — for a bf16 value that is bits 7..14 of its pattern.
__global__ void __launch_bounds__(256) group_scale_bytes_identity(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                                                  uint8_t* scales) {
  griddep_wait();
  const int64_t ng = K >> 5, total = M * ng;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / ng, g = i - row * ng;
    const uint32_t ef = group_max_mag(x, row, ldx, g) >> 7;
    scales[i] = (uint8_t)(ef > 2u ? ef - 2u : 0u);
  }
}

__global__ void __launch_bounds__(512) magnitude_histogram(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                                           unsigned long long* hist) {
  extern __shared__ uint32_t local[];                 // kMagBins counters
  for (int i = threadIdx.x; i < kMagBins; i += blockDim.x) local[i] = 0u;
  __syncthreads();
  griddep_wait();
  const int64_t chunks_per_row = K >> 3, total = M * chunks_per_row;    // 16-byte chunks
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / chunks_per_row, c = i - row * chunks_per_row;
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(x + row * ldx + c * 8));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      atomicAdd(&local[w[j] & 0x7FFFu], 1u);
      atomicAdd(&local[(w[j] >> 16) & 0x7FFFu], 1u);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < kMagBins; i += blockDim.x)
    if (local[i]) atomicAdd(&hist[i], (unsigned long long)local[i]);
}

// The k-th largest magnitude: the largest pattern t with count(patterns >= t) >= k.  One CTA of 1024
// threads; thread i owns the 32 patterns [32 i, 32 i + 32).  info[0] = t, info[1] = 0, info[2..3] = k.
__global__ void __launch_bounds__(1024) find_threshold(const unsigned long long* hist, unsigned long long k, uint32_t* info) {
  __shared__ unsigned long long part[1024];
  __shared__ int owner;
  griddep_wait();
  unsigned long long mine = 0;
  for (int j = 0; j < 32; ++j) mine += hist[threadIdx.x * 32 + j];
  part[threadIdx.x] = mine;
  if (threadIdx.x == 0) owner = 0;
  __syncthreads();
  // inclusive suffix sums over the 1024 partial counts (Hillis-Steele)
  for (int d = 1; d < 1024; d <<= 1) {
    const unsigned long long add = (threadIdx.x + d < 1024) ? part[threadIdx.x + d] : 0ull;
    __syncthreads();
    part[threadIdx.x] += add;
    __syncthreads();
  }
  // the owner is the highest thread whose suffix count reaches k
  const unsigned long long above = (threadIdx.x + 1 < 1024) ? part[threadIdx.x + 1] : 0ull;
  if (part[threadIdx.x] >= k && above < k) owner = (int)threadIdx.x + 1;
  __syncthreads();
  if ((int)threadIdx.x + 1 == owner) {
    unsigned long long run = above;
    uint32_t t = threadIdx.x * 32;
    for (int j = 31; j >= 0; --j) {
      run += hist[threadIdx.x * 32 + j];
      if (run >= k) { t = threadIdx.x * 32 + j; break; }
    }
    info[0] = t;
    info[1] = 0u;
    info[2] = (uint32_t)(k & 0xFFFFFFFFull);
    info[3] = (uint32_t)(k >> 32);
  }
  if (owner == 0 && threadIdx.x == 0) {                 // fewer than k entries in total: everything counts
    info[0] = 0u; info[1] = 0u; info[2] = (uint32_t)(k & 0xFFFFFFFFull); info[3] = (uint32_t)(k >> 32);
  }
}

__global__ void __launch_bounds__(256) outlier_group_mask(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                                          const uint32_t* info, uint8_t* mask) {
  griddep_wait();
  const uint32_t t = info[0];
  const int64_t ng = K >> 5, total = M * ng;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / ng, g = i - row * ng;
    mask[i] = group_max_mag(x, row, ldx, g) >= t ? 1 : 0;
  }
}

__global__ void __launch_bounds__(256) scale_histogram(const uint8_t* scales, const uint8_t* mask, int64_t n,
                                                       unsigned long long* hist) {
  __shared__ uint32_t local[512];
  for (int i = threadIdx.x; i < 512; i += blockDim.x) local[i] = 0u;
  __syncthreads();
  griddep_wait();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    atomicAdd(&local[(mask[i] ? 256 : 0) + scales[i]], 1u);
  __syncthreads();
  for (int i = threadIdx.x; i < 512; i += blockDim.x)
    if (local[i]) atomicAdd(&hist[i], (unsigned long long)local[i]);
}

__global__ void __launch_bounds__(256) scale_inflation(const uint8_t* before, const uint8_t* after, const uint8_t* mask,
                                                       int64_t n, unsigned long long* counts) {
  __shared__ uint32_t local[6];
  if (threadIdx.x < 6) local[threadIdx.x] = 0u;
  __syncthreads();
  griddep_wait();
  uint32_t mine[6] = {0, 0, 0, 0, 0, 0};
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int j = after[i] < before[i] ? 0 : (after[i] == before[i] ? 1 : 2);
    const int c = (mask[i] ? 3 : 0) + j;
#pragma unroll
    for (int q = 0; q < 6; ++q) mine[q] += (q == c) ? 1u : 0u;
  }
#pragma unroll
  for (int q = 0; q < 6; ++q) {
    uint32_t v = mine[q];
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    if ((threadIdx.x & 31) == 0 && v) atomicAdd(&local[q], v);
  }
  __syncthreads();
  if (threadIdx.x < 6 && local[threadIdx.x]) atomicAdd(&counts[threadIdx.x], (unsigned long long)local[threadIdx.x]);
}

inline unsigned grid_for(int64_t items, int threads, int sm_count, int per_sm) {
  const int64_t want = (items + threads - 1) / threads;
  const int64_t cap = (int64_t)sm_count * per_sm;
  return (unsigned)(want < 1 ? 1 : (want < cap ? want : cap));
}

}  // namespace stats
}  // namespace bro
