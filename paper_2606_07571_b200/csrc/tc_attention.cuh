// Tensor-core attention path (placeholder until the tcgen05 kernel lands).
#pragma once
#include "common.cuh"
#include "simt_kernels.cuh"
namespace bicache {
constexpr bool kTensorPathBuilt = false;
inline cudaError_t configure_tc_attention() { return cudaSuccess; }
inline cudaError_t launch_tc_attention(const ScheduleView&, const PoolView&, const TensorArgs&, int*, cudaStream_t) {
  return cudaErrorNotSupported;
}
}  // namespace bicache
