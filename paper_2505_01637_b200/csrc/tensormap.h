// Host-side creation of TMA tensor maps through the driver entry point (the library
// links only the CUDA runtime).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace morello {

// A rank-3 map over a dense row-major tensor [d2][d1][d0] (d0 innermost) of
// `elem_bytes`-byte elements with box {box0, box1, 1} and the given swizzle.
// Requirements (checked by the driver): base 16-byte aligned, d0 * elem_bytes a
// multiple of 16, box0 * elem_bytes <= the swizzle span.
cudaError_t make_tensor_map_3d(CUtensorMap* out, CUtensorMapDataType dtype, int elem_bytes,
                               const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                               uint32_t box0, uint32_t box1, CUtensorMapSwizzle swizzle,
                               CUtensorMapL2promotion promotion = CU_TENSOR_MAP_L2_PROMOTION_L2_256B);

}  // namespace morello
