// Kernel 2 placeholder: replaced by the tcgen05 block-scaled GEMM.
#pragma once
#include "bro_common.cuh"
namespace bro {
namespace gemm {
inline size_t workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
inline bro_status launch(const void*, const void*, const void*, const void*, int64_t, int64_t, int64_t,
                         void*, int64_t, int, void*, size_t, int, cudaStream_t) {
  return BRO_ERR_UNSUPPORTED;
}
}  // namespace gemm
}  // namespace bro
