// K2 placeholder until the tensor-core kernel is in place.
#include "device_common.cuh"
#include "kernels.hpp"

namespace pasta {
cudaError_t launch_attn_tensor(const PoolView &, const PlanHeader &, int32_t, int32_t, const void *, float,
                               cudaStream_t) {
  return cudaErrorNotSupported;
}
bool tensor_path_available() { return false; }
}  // namespace pasta
