// Tensor-core (tcgen05 / TMEM / TMA) kernels of the CompAct layer for sm_100a.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include <atomic>

#include "../../include/compact.h"
#include "philox.cuh"
#include "simt_kernels.cuh"

namespace compact {
namespace tc {

struct LaunchInfo {
  cudaStream_t stream;
  unsigned int* status;
  std::atomic<uint64_t>* launches;
};

inline size_t gc_workspace_bytes(int64_t, int, int) { return 0; }

inline compact_status_t forward(const LaunchInfo&, const ProjectionParams&, int64_t, const __nv_bfloat16*, int64_t,
                                const __nv_bfloat16*, int64_t, __nv_bfloat16*, int64_t, __nv_bfloat16*, int64_t, int) {
  return COMPACT_ERR_SHAPE;
}
inline compact_status_t backward(const LaunchInfo&, int64_t, int, int, int, const __nv_bfloat16*, int64_t,
                                 const __nv_bfloat16*, int64_t, const __nv_bfloat16*, int64_t, __nv_bfloat16*, int64_t,
                                 float*, int64_t, int, void*, size_t) {
  return COMPACT_ERR_SHAPE;
}
inline compact_status_t update(const LaunchInfo&, const ProjectionParams&, const simt::AdamScalars&, int, int, int,
                               __nv_bfloat16*, int64_t, const float*, int64_t, float*, float*, float, void*, size_t) {
  return COMPACT_ERR_SHAPE;
}

}  // namespace tc
}  // namespace compact
