// Skinny MatmulAccum: C[b, 0:m, :] += A[b, 0:m, :] x B[b] for m <= 16 on the
// FP32 FMA units, streaming B from HBM exactly once.
//
// Decomposition.  The n columns are cut into "units" of VEC columns (one
// 2*VEC-byte load).  A thread block owns `units` adjacent units and one slice
// of the k range; its threads form a (row_lanes x units) grid: thread
// (r, u) visits rows r, r + row_lanes, ... of the slice and keeps M x VEC f32
// accumulators for unit u.  A warp therefore reads contiguous 2*VEC*units-byte
// row segments, and every thread has UNROLL independent loads in flight.
// The rows of A that the slice needs sit in shared memory as f32, transposed to
// [k][M] so that one thread reads its M multipliers with vector loads.
// At the end the row lanes are summed through shared memory in a fixed order
// (lane 0, 1, 2, ...), so results are deterministic.  With one k slice the
// block adds its sums to C itself; with several it writes them to
// partial[slice][b][m][n] and reduce_kernel adds the slices in slice order and
// then adds C once.
//
// Flat form (FLAT, 16-byte loads only): when n % 8 != 0 or B is not 16-byte aligned, the rows
// of B start at varying offsets inside their 16-byte granules and the plain form falls back
// to 8-, 4- or 2-byte loads, several times slower.  Instead every thread loads ALIGNED
// 16-byte granules: for row p and column block cb, granule ul of the thread block starts d
// elements before column cb * W + 8 ul, d = the offset of (p, cb * W) inside its granule.
// d depends only on p mod 8 (8 rows of n elements shift by whole granules), and a thread's
// rows are 8 | row_lanes apart, so d is a constant of the thread: its 8 accumulators simply
// belong to columns shifted left by d.  A block carries one granule more than its W / 8
// (columns W .. W + 7 - d of the shifted windows), the final sum over the row lanes reads
// lane r's value of column x at index x + d_r, and accumulators of columns outside [0, n)
// (the neighbouring rows' elements a granule also holds) are never read.  Loads stay inside
// the 16-byte granules that hold bytes of B.
#include <algorithm>

#include "internal.h"

namespace morello {
namespace {

constexpr int kSmemABudget = 64 * 1024;  // bytes of shared memory for the staged rows of A

struct SkinnyParams {
  const uint16_t* A;
  const uint16_t* B;
  float* C;
  float* partial;
  int64_t a_batch, b_batch, c_batch;  // batch strides in elements
  int64_t k, n;
  int64_t k_per_split;
  int64_t partial_split_stride;  // b * m * n
  int m;
  int num_units;  // n / VEC
  int units;
  int row_lanes;
  int col_blocks;
  int split_k;
  int k_chunk;
  int overwrite;  // 1: C = sum instead of C += sum
  int flat_cols;  // flat form: output columns per thread block, 8 * (units - 1)
};

template <int M_T>
struct Tuning;
template <> struct Tuning<1>  { static constexpr int kThreads = 1024, kUnroll = 8; };
template <> struct Tuning<2>  { static constexpr int kThreads = 1024, kUnroll = 8; };
template <> struct Tuning<4>  { static constexpr int kThreads = 512,  kUnroll = 8; };
template <> struct Tuning<8>  { static constexpr int kThreads = 512,  kUnroll = 4; };
template <> struct Tuning<16> { static constexpr int kThreads = 256,  kUnroll = 4; };

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Streaming loads of B: read-only path, no L1 allocation (every byte is used once).
template <int VEC>
struct BVec;
template <> struct BVec<8> {
  uint32_t w[4];
  __device__ __forceinline__ void load(const uint16_t* p) {
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p));
  }
  __device__ __forceinline__ float get(int j) const { return (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]); }
};
template <> struct BVec<4> {
  uint32_t w[2];
  __device__ __forceinline__ void load(const uint16_t* p) {
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];"
                 : "=r"(w[0]), "=r"(w[1]) : "l"(p));
  }
  __device__ __forceinline__ float get(int j) const { return (j & 1) ? bf16_hi(w[j >> 1]) : bf16_lo(w[j >> 1]); }
};
template <> struct BVec<2> {
  uint32_t w[1];
  __device__ __forceinline__ void load(const uint16_t* p) {
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p));
  }
  __device__ __forceinline__ float get(int j) const { return (j & 1) ? bf16_hi(w[0]) : bf16_lo(w[0]); }
};
template <> struct BVec<1> {
  uint16_t h;
  __device__ __forceinline__ void load(const uint16_t* p) {
    asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(h) : "l"(p));
  }
  __device__ __forceinline__ float get(int) const { return __uint_as_float(((uint32_t)h) << 16); }
};

template <int M_T, int VEC>
__device__ __forceinline__ void fma_row(float (&acc)[M_T][VEC], const float* __restrict__ a_row,
                                        const BVec<VEC>& v) {
  float a[M_T];
  if constexpr (M_T >= 4) {
#pragma unroll
    for (int i = 0; i < M_T; i += 4) {
      const float4 q = *reinterpret_cast<const float4*>(a_row + i);
      a[i] = q.x; a[i + 1] = q.y; a[i + 2] = q.z; a[i + 3] = q.w;
    }
  } else if constexpr (M_T == 2) {
    const float2 q = *reinterpret_cast<const float2*>(a_row);
    a[0] = q.x; a[1] = q.y;
  } else {
    a[0] = a_row[0];
  }
#pragma unroll
  for (int j = 0; j < VEC; ++j) {
    const float bj = v.get(j);
#pragma unroll
    for (int i = 0; i < M_T; ++i) acc[i][j] = fmaf(a[i], bj, acc[i][j]);
  }
}

// Programmatic dependent launch: a kernel launched with the stream-serialisation
// attribute may start while its predecessor drains; it must not touch global
// memory before pdl_wait() returns (the predecessor has then completed and its
// writes are visible).  pdl_release() lets the successor's blocks be scheduled.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;"); }

template <int M_T, int VEC, int UNROLL, int THREADS, bool FLAT = false>
__global__ void __launch_bounds__(THREADS)
skinny_kernel(const SkinnyParams p) {
  static_assert(!FLAT || VEC == 8, "the flat form loads whole 16-byte granules");
  extern __shared__ __align__(16) float smem[];
  float* a_s = smem;                                  // [k_chunk][M_T]
  float* red = smem + (size_t)p.k_chunk * M_T;        // [row_lanes][M_T * units * VEC]

  const int t = threadIdx.x;
  const int ul = t % p.units;
  const int rl = t / p.units;
  const int cb = blockIdx.x % p.col_blocks;
  const int s = blockIdx.x / p.col_blocks;
  const int bb = blockIdx.y;
  const int unit = cb * p.units + ul;
  const int64_t k0 = (int64_t)s * p.k_per_split;
  const int64_t k1 = min(p.k, k0 + p.k_per_split);
  const int R = p.row_lanes;
  const int64_t step = (int64_t)R * p.n;

  float acc[M_T][VEC];
#pragma unroll
  for (int i = 0; i < M_T; ++i)
#pragma unroll
    for (int j = 0; j < VEC; ++j) acc[i][j] = 0.f;

  const uint16_t* a_base = p.A + (int64_t)bb * p.a_batch;
  // Element index (address / 2) of (row 0 of the batch, first column of this column block).
  const uint64_t flat_e0 = (reinterpret_cast<uint64_t>(p.B) >> 1) + (uint64_t)bb * p.b_batch +
                           (uint64_t)cb * p.flat_cols;
  // First column of the thread's accumulators: plain form unit * VEC; flat form the column
  // block's first column, back by this row lane's offset d, plus 8 ul.
  int64_t col_off = (int64_t)unit * VEC;
  bool active = (rl < p.row_lanes) && (unit < p.num_units);
  if constexpr (FLAT) {
    const int d = (int)((flat_e0 + (uint64_t)(k0 + rl) * p.n) & 7u);
    col_off = (int64_t)cb * p.flat_cols - d + 8 * ul;
    active = (rl < p.row_lanes) && col_off < p.n;
  }
  const uint16_t* bp = p.B + (int64_t)bb * p.b_batch + col_off + (k0 + rl) * p.n;

  // The first group of B rows is requested before A is staged, so that the staging
  // latency hides under the first HBM round trip.  Nothing is touched before pdl_wait().
  BVec<VEC> v[UNROLL];
  bool preloaded = false;
  pdl_wait();
  if (active) {
    const int kcl0 = (int)min((int64_t)p.k_chunk, k1 - k0);
#pragma unroll
    for (int u = 0; u < UNROLL; ++u)
      if (rl + u * R < kcl0) v[u].load(bp + u * step);
    preloaded = true;
  }
  pdl_release();

  for (int64_t kc0 = k0; kc0 < k1; kc0 += p.k_chunk) {
    const int kcl = (int)min((int64_t)p.k_chunk, k1 - kc0);
    if (kc0 != k0) __syncthreads();  // previous chunk's readers are done with a_s
#pragma unroll
    for (int i = 0; i < M_T; ++i) {
      for (int q = t; q < kcl; q += blockDim.x) {
        const float av = (i < p.m)
            ? __uint_as_float(((uint32_t)a_base[(int64_t)i * p.k + kc0 + q]) << 16) : 0.f;
        a_s[q * M_T + i] = av;
      }
    }
    __syncthreads();
    if (active) {
      // Rows q, q + R, ... of the chunk in groups of UNROLL: all loads of a group are
      // issued before the first is consumed; rows past the chunk are predicated off.
      for (int q = rl; q < kcl; q += UNROLL * R) {
        if (!preloaded) {
#pragma unroll
          for (int u = 0; u < UNROLL; ++u)
            if (q + u * R < kcl) v[u].load(bp + u * step);
        }
        preloaded = false;
        bp += UNROLL * step;
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
          if (q + u * R < kcl) fma_row<M_T, VEC>(acc, a_s + (q + u * R) * M_T, v[u]);
      }
      // bp now points UNROLL*R-aligned past the chunk; rebase to the next chunk's first row.
      bp = p.B + (int64_t)bb * p.b_batch + col_off + (kc0 + kcl + rl) * p.n;
    }
  }

  // Sum the row lanes in lane order through shared memory.
  const int W = M_T * p.units * VEC;  // floats per row lane
  if (active) {
    float* dst = red + (size_t)rl * W + ul * VEC;
#pragma unroll
    for (int i = 0; i < M_T; ++i)
#pragma unroll
      for (int j = 0; j < VEC; ++j) dst[i * p.units * VEC + j] = acc[i][j];
  }
  __syncthreads();
  if constexpr (FLAT) {
    // Row lane r holds column x of this block at index x + d_r of its row of sums.
    const int cols = p.flat_cols;
    const int pitch = p.units * VEC;
    for (int o = t; o < M_T * cols; o += blockDim.x) {
      const int i = o / cols, x = o - i * cols;
      const int64_t col = (int64_t)cb * cols + x;
      if (i >= p.m || col >= p.n) continue;
      float sum = 0.f;
      for (int r = 0; r < R; ++r) {
        const int d = (int)((flat_e0 + (uint64_t)(k0 + r) * p.n) & 7u);
        const float v = red[(size_t)r * W + i * pitch + x + d];
        sum = r == 0 ? v : sum + v;
      }
      if (p.split_k == 1) {
        float* c = p.C + (int64_t)bb * p.c_batch + (int64_t)i * p.n + col;
        *c = p.overwrite ? sum : *c + sum;
      } else {
        p.partial[(int64_t)s * p.partial_split_stride + ((int64_t)bb * p.m + i) * p.n + col] = sum;
      }
    }
    return;
  }
  const int cols_here = p.units * VEC;
  const int64_t col_base = (int64_t)cb * cols_here;
  for (int o = t; o < W; o += blockDim.x) {
    const int i = o / cols_here;
    const int64_t col = col_base + (o - i * cols_here);
    if (i >= p.m || col >= p.n) continue;
    float sum = red[o];
    for (int r = 1; r < R; ++r) sum += red[(size_t)r * W + o];
    if (p.split_k == 1) {
      float* c = p.C + (int64_t)bb * p.c_batch + (int64_t)i * p.n + col;
      *c = p.overwrite ? sum : *c + sum;
    } else {
      p.partial[(int64_t)s * p.partial_split_stride + ((int64_t)bb * p.m + i) * p.n + col] = sum;
    }
  }
}

// C[b, i, :] += sum over slices, slice order fixed; one thread per output element.
__global__ void __launch_bounds__(256)
reduce_kernel(const float* __restrict__ partial, float* __restrict__ C, int64_t total,
              int64_t mn, int64_t c_batch, int split_k, int overwrite) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  pdl_wait();
  pdl_release();
  if (idx >= total) return;
  float sum = partial[idx];
  for (int s = 1; s < split_k; ++s) sum += partial[(int64_t)s * total + idx];
  const int64_t bb = idx / mn;
  float* c = C + bb * c_batch + (idx - bb * mn);
  *c = overwrite ? sum : *c + sum;
}

// The same sums, four neighbouring outputs per thread (shapes whose batch sizes and pointers
// keep every group of four inside one batch and 16-byte aligned).
__global__ void __launch_bounds__(256)
reduce4_kernel(const float4* __restrict__ partial, float* __restrict__ C, int64_t total4,
               int64_t mn, int64_t c_batch, int split_k, int overwrite) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  pdl_wait();
  pdl_release();
  if (idx >= total4) return;
  float4 sum = partial[idx];
  for (int s = 1; s < split_k; ++s) {
    const float4 v = partial[(int64_t)s * total4 + idx];
    sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
  }
  const int64_t e = idx * 4;
  const int64_t bb = e / mn;
  float4* c = reinterpret_cast<float4*>(C + bb * c_batch + (e - bb * mn));
  if (!overwrite) {
    const float4 v = *c;
    sum.x = v.x + sum.x; sum.y = v.y + sum.y; sum.z = v.z + sum.z; sum.w = v.w + sum.w;
  }
  *c = sum;
}

// The same sums when C has fewer columns than the partial sums (zero-padded operands): C is dense
// [rows][c_cols], the partial sums are [split_k][rows][n]; one thread per element of C.
__global__ void __launch_bounds__(256)
reduce_narrow_kernel(const float* __restrict__ partial, float* __restrict__ C, int64_t rows, int64_t n,
                     int64_t c_cols, int split_k, int overwrite) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  pdl_wait();
  pdl_release();
  if (idx >= rows * c_cols) return;
  const int64_t r = idx / c_cols, j = idx - r * c_cols;
  const float* src = partial + r * n + j;
  float sum = src[0];
  for (int s = 1; s < split_k; ++s) sum += src[(int64_t)s * rows * n];
  C[idx] = overwrite ? sum : C[idx] + sum;
}

// Launch with programmatic stream serialisation (see pdl_wait above).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, int threads, size_t smem,
                       cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

template <int M_T, int VEC>
cudaError_t launch_one(const SkinnyPlan& plan, const SkinnyParams& prm, int64_t b,
                       cudaStream_t stream) {
  auto kern = skinny_kernel<M_T, VEC, Tuning<M_T>::kUnroll, Tuning<M_T>::kThreads>;
  if (plan.smem_bytes > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)plan.smem_bytes);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)(plan.col_blocks * plan.split_k), (unsigned)b, 1);
  return launch_pdl(kern, grid, plan.threads, plan.smem_bytes, stream, prm);
}

template <int M_T>
cudaError_t launch_flat(const SkinnyPlan& plan, const SkinnyParams& prm, int64_t b,
                        cudaStream_t stream) {
  auto kern = skinny_kernel<M_T, 8, Tuning<M_T>::kUnroll, Tuning<M_T>::kThreads, true>;
  if (plan.smem_bytes > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)plan.smem_bytes);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((unsigned)(plan.col_blocks * plan.split_k), (unsigned)b, 1);
  return launch_pdl(kern, grid, plan.threads, plan.smem_bytes, stream, prm);
}

template <int M_T>
cudaError_t launch_vec(const SkinnyPlan& plan, const SkinnyParams& prm, int64_t b,
                       cudaStream_t stream) {
  if (plan.flat) return launch_flat<M_T>(plan, prm, b, stream);
  switch (plan.vec) {
    case 8: return launch_one<M_T, 8>(plan, prm, b, stream);
    case 4: return launch_one<M_T, 4>(plan, prm, b, stream);
    case 2: return launch_one<M_T, 2>(plan, prm, b, stream);
    default: return launch_one<M_T, 1>(plan, prm, b, stream);
  }
}

int max_threads_for(int m_tile) {
  switch (m_tile) {
    case 1: return Tuning<1>::kThreads;
    case 2: return Tuning<2>::kThreads;
    case 4: return Tuning<4>::kThreads;
    case 8: return Tuning<8>::kThreads;
    default: return Tuning<16>::kThreads;
  }
}

}  // namespace

int skinny_vec(int64_t n, const void* B) {
  const uintptr_t addr = reinterpret_cast<uintptr_t>(B);
  for (int vec = 8; vec > 1; vec >>= 1)
    if (n % vec == 0 && addr % (2 * vec) == 0) return vec;
  return 1;
}

namespace {

SkinnyPlan plan_impl(int sms, int64_t b, int m, int64_t k, int64_t n, int vec, int split_k, bool flat) {
  SkinnyPlan pl{};
  pl.m_tile = m <= 1 ? 1 : m <= 2 ? 2 : m <= 4 ? 4 : m <= 8 ? 8 : 16;
  pl.flat = flat;
  if (flat) vec = 8;
  pl.vec = vec;
  int max_threads = max_threads_for(pl.m_tile);
  const int64_t num_units = flat ? (n + 7) / 8 : n / vec;
  const int unit_cap = (int)std::min<int64_t>(num_units, 128 / vec);  // <= 256-byte row segments
  // One wave of thread blocks over the SMs when the columns allow it.
  const int64_t per_sm = (b * num_units + sms - 1) / sms;
  int units;
  if (per_sm <= unit_cap) {
    units = (int)std::max<int64_t>(per_sm, 1);
  } else {
    const int64_t waves = (per_sm + unit_cap - 1) / unit_cap;
    units = (int)((per_sm + waves - 1) / waves);
  }
  units = std::min<int>(units, unit_cap);
  pl.col_blocks = (int)((num_units + units - 1) / units);
  if (flat) ++units;   // the granule that holds the shifted windows' last columns
  pl.units = units;
  const int64_t blocks = b * pl.col_blocks;
  int s = split_k;
  if (s <= 0) {
    s = 1;
    if (blocks * 2 <= sms && k >= 512)
      s = (int)std::min<int64_t>(std::min<int64_t>(sms / blocks, k / 256), 32);
  }
  s = (int)std::max<int64_t>(1, std::min<int64_t>(s, std::max<int64_t>(k, 1)));
  int64_t kps = (std::max<int64_t>(k, 1) + s - 1) / s;
  kps = (kps + 7) / 8 * 8;
  pl.k_per_split = kps;
  pl.split_k = (int)((std::max<int64_t>(k, 1) + kps - 1) / kps);
  // More thread blocks than SMs with a single row: blocks of 512 threads, so that two share an
  // SM instead of running in two rounds (with at most one block per SM the full 1024 threads
  // are better).
  if (pl.m_tile == 1 && blocks * pl.split_k > sms) max_threads = std::min(max_threads, 512);
  // Row lanes: as many as the thread budget allows, a multiple of 8 when possible,
  // never more than the slice has rows.
  int rows = max_threads / units;
  if (rows >= 8) rows = rows / 8 * 8;
  rows = (int)std::max<int64_t>(1, std::min<int64_t>(rows, kps));
  pl.row_lanes = rows;
  pl.threads = (rows * units + 31) / 32 * 32;
  pl.k_chunk = (int)std::min<int64_t>(kps, kSmemABudget / (4 * pl.m_tile));
  pl.smem_bytes = (size_t)pl.k_chunk * pl.m_tile * 4 +
                  (size_t)rows * pl.m_tile * units * vec * 4;
  pl.workspace_bytes = pl.split_k > 1 ? (size_t)pl.split_k * b * m * n * 4 : 0;
  return pl;
}

}  // namespace

SkinnyPlan skinny_plan(int sms, int64_t b, int m, int64_t k, int64_t n, int vec, int split_k) {
  // Loads narrower than 16 bytes: the flat form (aligned granules, shifted columns) instead,
  // once there is a stream of B worth it.  It needs row lanes in multiples of 8.
  if (vec < 8 && k >= 64 && n >= 16) {
    const SkinnyPlan flat = plan_impl(sms, b, m, k, n, 8, split_k, true);
    if (flat.row_lanes % 8 == 0) return flat;
  }
  return plan_impl(sms, b, m, k, n, vec, split_k, false);
}

cudaError_t skinny_launch(const SkinnyPlan& plan, int64_t b, int m, int64_t k, int64_t n,
                          const uint16_t* A, int64_t a_batch, const uint16_t* B, float* C,
                          int64_t c_batch, float* workspace, cudaStream_t stream,
                          uint64_t* launches, bool overwrite) {
  SkinnyParams prm{};
  prm.overwrite = overwrite ? 1 : 0;
  prm.A = A; prm.B = B; prm.C = C; prm.partial = workspace;
  prm.a_batch = a_batch; prm.b_batch = k * n; prm.c_batch = c_batch;
  prm.k = k; prm.n = n;
  prm.k_per_split = plan.k_per_split;
  prm.partial_split_stride = b * m * n;
  prm.m = m;
  prm.num_units = (int)(n / plan.vec);
  prm.flat_cols = plan.flat ? 8 * (plan.units - 1) : 0;
  prm.units = plan.units;
  prm.row_lanes = plan.row_lanes;
  prm.col_blocks = plan.col_blocks;
  prm.split_k = plan.split_k;
  prm.k_chunk = plan.k_chunk;
  // grid.y carries the batch index; larger batches go in slabs.
  for (int64_t b0 = 0; b0 < b; b0 += 65535) {
    const int64_t bn = std::min<int64_t>(65535, b - b0);
    SkinnyParams q = prm;
    q.A = A + b0 * a_batch; q.B = B + b0 * k * n; q.C = C + b0 * c_batch;
    q.partial = workspace ? workspace + b0 * m * n : nullptr;
    cudaError_t e;
    switch (plan.m_tile) {
      case 1: e = launch_vec<1>(plan, q, bn, stream); break;
      case 2: e = launch_vec<2>(plan, q, bn, stream); break;
      case 4: e = launch_vec<4>(plan, q, bn, stream); break;
      case 8: e = launch_vec<8>(plan, q, bn, stream); break;
      default: e = launch_vec<16>(plan, q, bn, stream); break;
    }
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  if (plan.split_k > 1) {
    cudaError_t e = skinny_reduce_launch(workspace, C, b, m, n, c_batch, plan.split_k, stream, overwrite);
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaSuccess;
}

namespace {

// One warp per output column j of one batch: lane l visits k = l, l + 32, ... of row j of Bt
// (coalesced) for every row i of A in turn.
__global__ void __launch_bounds__(256)
colmajor_fallback_kernel(const uint16_t* __restrict__ A, const uint16_t* __restrict__ Bt,
                         float* __restrict__ C, int64_t m, int64_t k, int64_t n, int overwrite) {
  const int lane = threadIdx.x & 31;
  const int64_t j = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t bb = blockIdx.y;
  if (j >= n) return;
  const uint16_t* brow = Bt + (bb * n + j) * k;
  for (int64_t i = 0; i < m; ++i) {
    const uint16_t* arow = A + (bb * m + i) * k;
    float sum = 0.f;
    for (int64_t p = lane; p < k; p += 32)
      sum = fmaf(__uint_as_float(((uint32_t)arow[p]) << 16), __uint_as_float(((uint32_t)brow[p]) << 16), sum);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (lane == 0) {
      float* c = C + (bb * m + i) * n + j;
      *c = overwrite ? sum : *c + sum;
    }
  }
}

}  // namespace

cudaError_t colmajor_fallback_launch(int64_t b, int64_t m, int64_t k, int64_t n, const uint16_t* A,
                                     const uint16_t* Bt, float* C, bool overwrite,
                                     cudaStream_t stream, uint64_t* launches) {
  for (int64_t b0 = 0; b0 < b; b0 += 65535) {
    const int64_t bn = std::min<int64_t>(65535, b - b0);
    dim3 grid((unsigned)((n + 7) / 8), (unsigned)bn, 1);
    colmajor_fallback_kernel<<<grid, 256, 0, stream>>>(A + b0 * m * k, Bt + b0 * n * k, C + b0 * m * n,
                                                       m, k, n, overwrite ? 1 : 0);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaSuccess;
}

namespace {

// Packed B where the tensor kernels cannot run: one thread per output column and (row, batch)
// pair taken in strides of the grid; neighbouring threads read neighbouring columns of a strip
// (coalesced inside a strip), k in increasing order.
__global__ void __launch_bounds__(256)
packed_fallback_kernel(const uint16_t* __restrict__ A, const uint16_t* __restrict__ Bp,
                       float* __restrict__ C, int64_t b, int64_t m, int64_t k, int64_t n,
                       int64_t strip, int overwrite) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const int64_t strips = (n + strip - 1) / strip;
  for (int64_t bb = blockIdx.z; bb < b; bb += gridDim.z) {
    const uint16_t* col = Bp + ((bb * strips + j / strip) * k) * strip + (j % strip);
    for (int64_t i = blockIdx.y; i < m; i += gridDim.y) {
      const uint16_t* arow = A + (bb * m + i) * k;
      float sum = 0.f;
      for (int64_t p = 0; p < k; ++p)
        sum = fmaf(__uint_as_float(((uint32_t)arow[p]) << 16),
                   __uint_as_float(((uint32_t)col[p * strip]) << 16), sum);
      float* c = C + (bb * m + i) * n + j;
      *c = overwrite ? sum : *c + sum;
    }
  }
}

}  // namespace

cudaError_t packed_fallback_launch(int64_t strip, int64_t b, int64_t m, int64_t k, int64_t n,
                                   const uint16_t* A, const uint16_t* Bp, float* C, bool overwrite,
                                   cudaStream_t stream, uint64_t* launches) {
  dim3 grid((unsigned)((n + 255) / 256), (unsigned)std::min<int64_t>(m, 65535),
            (unsigned)std::min<int64_t>(b, 65535));
  packed_fallback_kernel<<<grid, 256, 0, stream>>>(A, Bp, C, b, m, k, n, strip, overwrite ? 1 : 0);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ++*launches;
  return cudaSuccess;
}

cudaError_t skinny_reduce_launch(const float* partial, float* C, int64_t b, int m, int64_t n,
                                 int64_t c_batch, int split_k, cudaStream_t stream, bool overwrite,
                                 int64_t c_cols) {
  if (c_cols > 0 && c_cols != n) {
    const int64_t rows = b * m, blocks = (rows * c_cols + 255) / 256;
    return launch_pdl(reduce_narrow_kernel, dim3((unsigned)blocks, 1, 1), 256, 0, stream, partial, C, rows, n,
                      c_cols, split_k, overwrite ? 1 : 0);
  }
  const int64_t total = b * m * n;
  const int64_t mn = (int64_t)m * n;
  if (mn % 4 == 0 && c_batch % 4 == 0 && reinterpret_cast<uintptr_t>(partial) % 16 == 0 &&
      reinterpret_cast<uintptr_t>(C) % 16 == 0) {
    const int64_t total4 = total / 4;
    return launch_pdl(reduce4_kernel, dim3((unsigned)((total4 + 255) / 256), 1, 1), 256, 0, stream,
                      reinterpret_cast<const float4*>(partial), C, total4, mn, c_batch, split_k,
                      overwrite ? 1 : 0);
  }
  const int64_t blocks = (total + 255) / 256;
  return launch_pdl(reduce_kernel, dim3((unsigned)blocks, 1, 1), 256, 0, stream, partial, C, total,
                    (int64_t)m * n, c_batch, split_k, overwrite ? 1 : 0);
}

}  // namespace morello
