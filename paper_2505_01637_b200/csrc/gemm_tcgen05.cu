// tcgen05 GEMM path (placeholder until the tensor-core kernel lands): reports every
// shape as unsupported so that the selector keeps to the skinny path.
#include "internal.h"

namespace morello {

bool gemm_shape_supported(int64_t, int64_t, int64_t, int64_t, const void*, const void*,
                          const void*) {
  return false;
}

GemmPlan gemm_plan(int, int64_t, int64_t, int64_t, int64_t, int) { return GemmPlan{false, 1, 0}; }

cudaError_t gemm_launch(const DeviceInfo&, const GemmPlan&, int64_t, int64_t, int64_t, int64_t,
                        const uint16_t*, const uint16_t*, float*, float*, cudaStream_t, uint64_t*) {
  return cudaErrorNotSupported;
}

}  // namespace morello
