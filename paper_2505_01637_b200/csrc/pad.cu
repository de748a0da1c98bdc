// Shapes the TMA engine cannot address (k % 8 != 0 or n % 8 != 0), with enough rows that the
// FP32-FMA kernels would stream B many times over: the operands are copied once into
// zero-padded, 16-byte-aligned buffers in the workspace,
//     A'[b][m][k8]  (k8 = k rounded up to 8; the added columns are zero),
//     B'[b][k8][n8] (n8 = n rounded up to 8; the added rows and columns are zero),
// by one launch, and the tensor-core kernels compute MatmulAccum(b, m, k8, n8) on them -- the
// zero padding adds exact zeros to every sum.  When C's rows cannot be addressed by the TMA
// engine either (n % 8 != 0 or a base that is not 16-byte aligned) the kernels' epilogues add
// their sums to the first n columns of each row of C straight from registers; C is still added
// exactly once, last, to the complete sum.
#include "internal.h"
#include "sm100.cuh"

namespace morello {
namespace {

// The copy launch and the tensor-core call form a chain of short launches: each is launched
// with programmatic stream serialisation, waits for its predecessor before it touches global
// memory and lets its successor's blocks be scheduled right away, so that the launch latencies
// overlap.  (Every kernel of the chain executes the wait, so "the predecessor has completed"
// carries through the whole chain.)
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kern)(KArgs...), unsigned blocks, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(blocks, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// dst[bb][r][c] = src[bb][r][c] inside the source extents, else 0; dst is [b][rows_out][cols_out]
// with cols_out % 8 == 0 and a 16-byte-aligned base.  One thread per 8 output elements.
struct PadJob {
  const uint16_t* src;
  uint4* dst;
  int64_t rows_in, cols_in, rows_out, cols_out;
  int64_t threads;   // b * rows_out * cols_out / 8; 0: nothing to copy
};

__device__ __forceinline__ void pad_one(const PadJob& j, int64_t idx) {
  const int64_t groups = j.cols_out / 8;
  const int64_t g = idx % groups;
  const int64_t r = (idx / groups) % j.rows_out;
  const int64_t bb = idx / (groups * j.rows_out);
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (r < j.rows_in) {
    const uint16_t* row = j.src + (bb * j.rows_in + r) * j.cols_in;
    const int64_t c0 = g * 8;
    const uint16_t* at = row + c0;
    if (c0 + 8 <= j.cols_in) {
      // Eight elements inside the row: 32-bit loads where the address allows (the source rows
      // are only 2-byte aligned), 4 or 5 loads instead of 8.  (Aligned 16-byte granules with a
      // funnel shift -- two loads per thread, or one load and the neighbour's granule by warp
      // shuffles -- were both measured slower.)
      if ((reinterpret_cast<uintptr_t>(at) & 2u) == 0) {
        const uint32_t* q = reinterpret_cast<const uint32_t*>(at);
        w[0] = q[0]; w[1] = q[1]; w[2] = q[2]; w[3] = q[3];
      } else {
        const uint32_t h0 = at[0], h7 = at[7];
        const uint32_t* q = reinterpret_cast<const uint32_t*>(at + 1);
        const uint32_t x0 = q[0], x1 = q[1], x2 = q[2];
        w[0] = h0 | (x0 << 16);
        w[1] = (x0 >> 16) | (x1 << 16);
        w[2] = (x1 >> 16) | (x2 << 16);
        w[3] = (x2 >> 16) | (h7 << 16);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t v = (c0 + e < j.cols_in) ? (uint32_t)at[e] : 0u;
        w[e >> 1] |= v << ((e & 1) * 16);
      }
    }
  }
  j.dst[idx] = make_uint4(w[0], w[1], w[2], w[3]);
}

// Both copies in one launch: threads [0, a.threads) pad A, the next b.threads pad B.
__global__ void __launch_bounds__(256)
pad_operands_kernel(const PadJob a, const PadJob b) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  sm100::pdl_wait();
  sm100::pdl_release();
  if (idx < a.threads) pad_one(a, idx);
  else if (idx - a.threads < b.threads) pad_one(b, idx - a.threads);
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

PadPlan pad_plan(int64_t b, int64_t m, int64_t k, int64_t n, const void* A, const void* B,
                 const void* C) {
  PadPlan p{};
  p.k8 = (k + 7) / 8 * 8;
  p.n8 = (n + 7) / 8 * 8;
  const bool k_odd = (k % 8) != 0, n_odd = (n % 8) != 0;
  p.stage_a = k_odd || reinterpret_cast<uintptr_t>(A) % 16 != 0;
  p.stage_b = k_odd || n_odd || reinterpret_cast<uintptr_t>(B) % 16 != 0;
  p.stage_c = n_odd || reinterpret_cast<uintptr_t>(C) % 16 != 0;
  p.bytes_a = p.stage_a ? round256((size_t)b * m * p.k8 * 2) : 0;
  p.bytes_b = p.stage_b ? round256((size_t)b * p.k8 * p.n8 * 2) : 0;
  return p;
}

cudaError_t pad_operands_launch(const PadPlan& p, int64_t b, int64_t m, int64_t k, int64_t n,
                                const uint16_t* A, const uint16_t* B, uint16_t* A_pad,
                                uint16_t* B_pad, cudaStream_t stream, uint64_t* launches) {
  PadJob ja{}, jb{};
  if (p.stage_a) ja = PadJob{A, reinterpret_cast<uint4*>(A_pad), m, k, m, p.k8, b * m * (p.k8 / 8)};
  if (p.stage_b) jb = PadJob{B, reinterpret_cast<uint4*>(B_pad), k, n, p.k8, p.n8, b * p.k8 * (p.n8 / 8)};
  const int64_t threads = ja.threads + jb.threads;
  if (threads == 0) return cudaSuccess;
  const int64_t blocks = (threads + 255) / 256;
  if (blocks >= (1ll << 31)) return cudaErrorInvalidValue;
  const cudaError_t e = launch_chained(pad_operands_kernel, (unsigned)blocks, stream, ja, jb);
  if (e != cudaSuccess) return e;
  ++*launches;
  return cudaSuccess;
}

}  // namespace morello
