// MatmulAccum on float32 inputs through the bf16 tensor-core kernels.
//
// A float is the exact sum of three bf16 values: x1 = bf16(x), x2 = bf16(x - x1),
// x3 = bf16(x - x1 - x2) (each difference is exact in float: every bf16 takes the next 8 of
// the 24 significant bits).  Then
//     a * b = sum over i, j of a_i * b_j,
// where a_i * b_j is about 2^(-8 (i + j - 2)) of a * b.  The six terms with i + j <= 4 are
// kept; the three dropped ones are below 2^-23 of |a * b|, well inside the acceptance rule
// (1e-5 of sum |a * b|).  Each kept term is a bf16 x bf16 product, exact in f32, which is
// what the tensor-core kernels accumulate.
//
// Rather than six calls, the six terms are laid side by side along k: the split kernels write
//     A6[b][m][6k] = [ A3 | A1 | A2 | A2 | A1 | A1 ]        (columns)
//     B6[b][6k][n] = [ B1 ; B3 ; B2 ; B1 ; B2 ; B1 ]        (rows)
// so that A6 x B6 = A3 B1 + A1 B3 + A2 B2 + A2 B1 + A1 B2 + A1 B1 (smallest terms first), and
// one ordinary MatmulAccum(b, m, 6k, n) on bf16 does the rest -- same kernels, same selector,
// C added once, deterministic.  Inputs whose values are bf16-exact (small integers, say) give
// A2 = A3 = 0 and the result is exact.
//
// When k is a whole number of the tensor kernels' 64-element blocks and the call goes to them,
// only the three terms are stored -- A3[b][m][3k] = [ A1 | A2 | A3 ], B3[b][3k][n] = [ B1 ; B2 ; B3 ]
// -- and the kernels read them as six segments of k in the order above (KSegments): the same
// products in the same order, half the bytes written here.
#include "internal.h"

namespace morello {
namespace {

__device__ __forceinline__ uint16_t bf16_rne(float x) {   // finite inputs
  const uint32_t u = __float_as_uint(x);
  return (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}
__device__ __forceinline__ float bf16_as_float(uint16_t h) { return __uint_as_float(((uint32_t)h) << 16); }

__device__ __forceinline__ void split3(float x, uint16_t& h1, uint16_t& h2, uint16_t& h3) {
  h1 = bf16_rne(x);
  const float r1 = x - bf16_as_float(h1);       // exact
  h2 = bf16_rne(r1);
  const float r2 = r1 - bf16_as_float(h2);      // exact
  h3 = bf16_rne(r2);
}

// A[rows][k] -> A6[rows][6k], blocks of k columns in the order 3, 1, 2, 2, 1, 1 -- or, kSix
// false, A3[rows][3k] in the order 1, 2, 3 (the kernels that read it then visit the stored
// terms in the six-term order themselves: KSegments).
template <bool kSix>
__global__ void __launch_bounds__(256)
split_a_kernel(const float* __restrict__ A, uint16_t* __restrict__ A6, int64_t rows, int64_t k) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * k) return;
  const int64_t r = idx / k, p = idx - r * k;
  uint16_t h1, h2, h3;
  split3(A[idx], h1, h2, h3);
  if constexpr (kSix) {
    uint16_t* row = A6 + r * 6 * k + p;
    row[0] = h3; row[k] = h1; row[2 * k] = h2; row[3 * k] = h2; row[4 * k] = h1; row[5 * k] = h1;
  } else {
    uint16_t* row = A6 + r * 3 * k + p;
    row[0] = h1; row[k] = h2; row[2 * k] = h3;
  }
}

// B[b][k][n] -> B6[b][6k][n], blocks of k rows in the order 1, 3, 2, 1, 2, 1 (kSix false:
// B3[b][3k][n], order 1, 2, 3).
template <bool kSix>
__global__ void __launch_bounds__(256)
split_b_kernel(const float* __restrict__ B, uint16_t* __restrict__ B6, int64_t b, int64_t k, int64_t n) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= b * k * n) return;
  const int64_t kn = k * n;
  const int64_t bb = idx / kn, rest = idx - bb * kn;      // rest = p * n + j
  uint16_t h1, h2, h3;
  split3(B[idx], h1, h2, h3);
  if constexpr (kSix) {
    uint16_t* dst = B6 + bb * 6 * kn + rest;
    dst[0] = h1; dst[kn] = h3; dst[2 * kn] = h2; dst[3 * kn] = h1; dst[4 * kn] = h2; dst[5 * kn] = h1;
  } else {
    uint16_t* dst = B6 + bb * 3 * kn + rest;
    dst[0] = h1; dst[kn] = h2; dst[2 * kn] = h3;
  }
}

// The same splits, eight neighbouring elements per thread: two 16-byte loads, six 16-byte
// stores (rows of A with k % 8 == 0, rows of B with n % 8 == 0, 16-byte-aligned pointers).
__device__ __forceinline__ void split8(const float4 lo, const float4 hi, uint4& t1, uint4& t2, uint4& t3) {
  const float x[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
  uint32_t w1[4], w2[4], w3[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    uint16_t a1, a2, a3, b1, b2, b3;
    split3(x[2 * e], a1, a2, a3);
    split3(x[2 * e + 1], b1, b2, b3);
    w1[e] = (uint32_t)a1 | ((uint32_t)b1 << 16);
    w2[e] = (uint32_t)a2 | ((uint32_t)b2 << 16);
    w3[e] = (uint32_t)a3 | ((uint32_t)b3 << 16);
  }
  t1 = make_uint4(w1[0], w1[1], w1[2], w1[3]);
  t2 = make_uint4(w2[0], w2[1], w2[2], w2[3]);
  t3 = make_uint4(w3[0], w3[1], w3[2], w3[3]);
}

template <bool kSix>
__global__ void __launch_bounds__(256)
split_a8_kernel(const float4* __restrict__ A, uint4* __restrict__ A6, int64_t rows, int64_t k8) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // group of 8 elements
  if (idx >= rows * k8) return;
  const int64_t r = idx / k8, g = idx - r * k8;
  uint4 t1, t2, t3;
  split8(A[2 * idx], A[2 * idx + 1], t1, t2, t3);
  if constexpr (kSix) {
    uint4* row = A6 + r * 6 * k8 + g;
    row[0] = t3; row[k8] = t1; row[2 * k8] = t2; row[3 * k8] = t2; row[4 * k8] = t1; row[5 * k8] = t1;
  } else {
    uint4* row = A6 + r * 3 * k8 + g;
    row[0] = t1; row[k8] = t2; row[2 * k8] = t3;
  }
}

template <bool kSix>
__global__ void __launch_bounds__(256)
split_b8_kernel(const float4* __restrict__ B, uint4* __restrict__ B6, int64_t b, int64_t kn8) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // group of 8 elements
  if (idx >= b * kn8) return;
  const int64_t bb = idx / kn8, rest = idx - bb * kn8;
  uint4 t1, t2, t3;
  split8(B[2 * idx], B[2 * idx + 1], t1, t2, t3);
  if constexpr (kSix) {
    uint4* dst = B6 + bb * 6 * kn8 + rest;
    dst[0] = t1; dst[kn8] = t3; dst[2 * kn8] = t2; dst[3 * kn8] = t1; dst[4 * kn8] = t2; dst[5 * kn8] = t1;
  } else {
    uint4* dst = B6 + bb * 3 * kn8 + rest;
    dst[0] = t1; dst[kn8] = t2; dst[2 * kn8] = t3;
  }
}

}  // namespace

size_t f32_split_bytes(int64_t b, int64_t m, int64_t k, int64_t n) {
  auto round256 = [](size_t x) { return (x + 255) / 256 * 256; };
  return round256((size_t)b * m * k * 12) + round256((size_t)b * k * n * 12);
}

namespace {

template <bool kSix>
cudaError_t split_launch(int64_t b, int64_t m, int64_t k, int64_t n, const float* A, const float* B,
                         uint16_t* A6, uint16_t* B6, cudaStream_t stream, uint64_t* launches) {
  const int64_t ea = b * m * k, eb = b * k * n;
  const bool a_vec = k % 8 == 0 && reinterpret_cast<uintptr_t>(A) % 16 == 0;
  const bool b_vec = n % 8 == 0 && reinterpret_cast<uintptr_t>(B) % 16 == 0;
  if (a_vec)
    split_a8_kernel<kSix><<<(unsigned)((ea / 8 + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(A), reinterpret_cast<uint4*>(A6), b * m, k / 8);
  else
    split_a_kernel<kSix><<<(unsigned)((ea + 255) / 256), 256, 0, stream>>>(A, A6, b * m, k);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ++*launches;
  if (b_vec)
    split_b8_kernel<kSix><<<(unsigned)((eb / 8 + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const float4*>(B), reinterpret_cast<uint4*>(B6), b, k * n / 8);
  else
    split_b_kernel<kSix><<<(unsigned)((eb + 255) / 256), 256, 0, stream>>>(B, B6, b, k, n);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ++*launches;
  return cudaSuccess;
}

}  // namespace

// `six`: the six-term layouts (any kernel can read them as a plain bf16 problem of 6k).  Else
// the three stored terms, for the kernels that take KSegments (k % 64 == 0).
cudaError_t f32_split_launch(int64_t b, int64_t m, int64_t k, int64_t n, const float* A, const float* B,
                             void* split, bool six, uint16_t** A6, uint16_t** B6, cudaStream_t stream,
                             uint64_t* launches) {
  auto round256 = [](size_t x) { return (x + 255) / 256 * 256; };
  *A6 = static_cast<uint16_t*>(split);
  *B6 = reinterpret_cast<uint16_t*>(static_cast<char*>(split) + round256((size_t)b * m * k * 12));
  return six ? split_launch<true>(b, m, k, n, A, B, *A6, *B6, stream, launches)
             : split_launch<false>(b, m, k, n, A, B, *A6, *B6, stream, launches);
}

}  // namespace morello
