// A self-test of the bounded waits: every mbarrier wait in the kernels of this library gives
// up after a time limit, records where in the device status word and lets the block return, so
// that a stalled pipeline ends as an error code instead of a hung device.  The kernel below
// exercises exactly that code path on purpose and harmlessly: one thread waits, with a short
// limit, on a barrier that nothing will ever arrive on, runs into the limit and returns.
#include "internal.h"
#include "sm100.cuh"

namespace morello {
namespace {

constexpr uint32_t kSelftestSite = 0x7e;   // site code in the status word

__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(uint32_t* status, uint64_t limit_ns, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    sm100::mbar_init(&bar, 1);
    abort_flag = 0;
    sm100::mbar_fence_init();
    // Phase 0 of a fresh barrier completes only after one arrival; none is ever made.
    const bool ok = sm100::mbar_wait(&bar, 0, &abort_flag, status, kSelftestSite, limit_ns);
    *gave_up = ok ? 0 : 1;
  }
}

}  // namespace

cudaError_t wait_timeout_selftest_launch(uint32_t* status, uint64_t limit_ns, int* gave_up,
                                         cudaStream_t stream) {
  wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns, gave_up);
  return cudaGetLastError();
}

}  // namespace morello
