// An entry point that never allocates: the split-k skinny kernel with its partial
// sums in a fixed device array that is part of the library image.
//
// Who needs it: callers that are not allowed to reach cudaMalloc at the time of the
// call -- a serving loop that has handed all device memory to its own pool (a late
// cudaMalloc could fail, and it would stall every stream of the process while it
// runs), or a component that is forbidden by policy from growing its footprint after
// start-up.  The ordinary entry points grow a per-device scratch buffer on demand;
// this one trades that for a hard size limit.
#include <algorithm>
#include <mutex>

#include "../../include/morello.h"
#include "internal.h"

namespace morello {
namespace {

constexpr size_t kStaticScratchBytes = MORELLO_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;
constexpr int kRowsPerLaunch = 16;

// Partial sums [split_k][b][rows][n] of the launch in flight.  Every GPU that loads
// the library carries this array until the process exits.  In host code this name is
// only a handle for cudaGetSymbolAddress -- it is not a device address.
static __device__ __align__(256) float g_static_scratch[kStaticScratchBytes / sizeof(float)];

struct NoAllocDevice {
  bool ready = false;
  int status = MORELLO_OK;
  int sms = 0;
  float* scratch = nullptr;  // device address of g_static_scratch on this device
};
NoAllocDevice g_noalloc[kMaxDevices];
std::mutex g_noalloc_mutex;

// First call on a device (that device being current): reads two device attributes and
// resolves the device address of the static array.  No allocation.
int noalloc_device(NoAllocDevice** out) {
  int dev = 0;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return record_cuda_error(ce);
  if (dev < 0 || dev >= kMaxDevices) return MORELLO_ERR_UNSUPPORTED_DEVICE;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  NoAllocDevice& st = g_noalloc[dev];
  if (!st.ready) {
    int major = 0, sms = 0;
    if ((ce = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess ||
        (ce = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
      return record_cuda_error(ce);
    st.sms = sms;
    if (major != 10) {
      st.status = MORELLO_ERR_UNSUPPORTED_DEVICE;
    } else {
      void* ptr = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (e != cudaSuccess || ptr == nullptr)   // not latched: a later call may try again
        return record_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
      st.scratch = static_cast<float*>(ptr);
      st.status = MORELLO_OK;
    }
    st.ready = true;
  }
  *out = &st;
  return st.status;
}

}  // namespace
}  // namespace morello

using namespace morello;

#pragma GCC visibility push(default)
extern "C" {

size_t morello_noalloc_scratch_limit(void) { return kStaticScratchBytes; }

int morello_matmul_accum_noalloc(int split_k, int64_t b, int64_t m, int64_t k, int64_t n,
                                 const void* A, const void* B, float* C, void* stream) {
  if (b < 0 || m < 0 || k < 0 || n < 0 || split_k < 0) return MORELLO_ERR_INVALID_SHAPE;
  int64_t mk, kn, mn, t;
  if (__builtin_mul_overflow(m, k, &mk) || __builtin_mul_overflow(k, n, &kn) ||
      __builtin_mul_overflow(m, n, &mn) || __builtin_mul_overflow(b, mk, &t) ||
      __builtin_mul_overflow(t, 2, &t) || __builtin_mul_overflow(b, kn, &t) ||
      __builtin_mul_overflow(t, 2, &t) || __builtin_mul_overflow(b, mn, &t) ||
      __builtin_mul_overflow(t, 4 * 64, &t))
    return MORELLO_ERR_INVALID_SHAPE;
  const bool empty = (b == 0 || m == 0 || n == 0 || k == 0);
  if (!empty) {
    if (!A || !B || !C) return MORELLO_ERR_NULL_POINTER;
    if (reinterpret_cast<uintptr_t>(A) % 2 || reinterpret_cast<uintptr_t>(B) % 2 ||
        reinterpret_cast<uintptr_t>(C) % 4)
      return MORELLO_ERR_MISALIGNED;
  }
  NoAllocDevice* st = nullptr;
  const int rc = noalloc_device(&st);
  if (rc != MORELLO_OK || empty) return rc;

  // Plan every row chunk first: nothing is enqueued unless all of them fit.
  const int vec = skinny_vec(n, B);
  for (int64_t i0 = 0; i0 < m; i0 += kRowsPerLaunch) {
    const int mc = (int)std::min<int64_t>(kRowsPerLaunch, m - i0);
    if (skinny_plan(st->sms, b, mc, k, n, vec, split_k).workspace_bytes > kStaticScratchBytes)
      return MORELLO_ERR_WORKSPACE;
  }
  const uint16_t* a = static_cast<const uint16_t*>(A);
  uint64_t launches = 0;
  for (int64_t i0 = 0; i0 < m; i0 += kRowsPerLaunch) {
    const int mc = (int)std::min<int64_t>(kRowsPerLaunch, m - i0);
    const SkinnyPlan plan = skinny_plan(st->sms, b, mc, k, n, vec, split_k);
    const cudaError_t e =
        skinny_launch(plan, b, mc, k, n, a + i0 * k, m * k, static_cast<const uint16_t*>(B),
                      C + i0 * n, m * n, st->scratch, static_cast<cudaStream_t>(stream), &launches);
    if (e != cudaSuccess) {
      count_launches(launches);
      return record_cuda_error(e);
    }
  }
  count_launches(launches);
  return MORELLO_OK;
}

}  // extern "C"
#pragma GCC visibility pop
