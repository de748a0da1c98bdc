// Streaming GEMV / very skinny MatmulAccum for sm_100a: C[b, 0:m, :] += A[b, 0:m, :] x B[b]
// for m <= 4 on the FP32 FMA units, with B brought in by the TMA engine.
//
// Decomposition.  The n columns are cut into strips of 64 (one 128-byte row segment of
// bf16) and, when the strips alone cannot fill the device or k is long, the k range into
// slices that are multiples of 128 rows.  One thread block owns one (batch, strip, slice):
//   warp 0      producer: one lane walks the slice in boxes of 128 k rows x 64 columns
//               (16 KiB), issuing TMA loads into a ring of 5 shared-memory stages, each
//               completing on the stage's "full" mbarrier;
//   warps 1-8   consumers: a warp reads 4 rows x 128 bytes per 16-byte-per-lane load, widens
//               bf16 to f32 (exact), multiplies by the rows' A values (the slice of A is
//               brought into shared memory once, by bulk copies when its alignment allows)
//               and accumulates 8 columns x m rows per lane with packed f32x2 FMAs; each warp
//               then frees the stage on its "empty" mbarrier.
// At the end the four row groups of a warp are added with shuffles and the eight warps
// through shared memory, always in the same order, so results are deterministic.  With one
// slice the block adds its sums to C (C was read early, the addition happens once, last).
// With 2, 4 or 8 slices the blocks of a strip form a thread-block cluster: each parks its
// sums in its own shared memory and block 0 reads them through distributed shared memory in
// slice order, adds C and stores -- one launch, no scratch, a fixed order.  More slices (a
// forced split) write partial[slice][b][m][n] for the slice-ordered reduce kernel.
//
// Between back-to-back calls.  The kernel is launched with programmatic stream
// serialisation.  Before griddepcontrol.wait it only sets up barriers and asks the TMA
// engine to prefetch its first boxes of B (and the lines of A) into L2 -- a prefetch moves
// nothing into the SM and cannot observe stale data, so it is legal before the preceding
// kernel has completed.  A block lets dependents launch when its producer has issued its
// last load: the next call's blocks then arrive while this call drains, and their
// prefetches keep HBM busy through this call's tail and the launch gap.  The ring (80 KiB)
// is sized so that at most two blocks share an SM: with three, the blocks of the crowded SMs
// finish microseconds after the rest.
//
// Rows of a box past k and columns past n are zero-filled by the TMA engine.  Every
// barrier wait is bounded; on a timeout the block records a status word and writes nothing.
#include <algorithm>
#include <mutex>

#include "internal.h"
#include "sm100.cuh"
#include "tensormap.h"

namespace morello {
namespace {

using namespace sm100;

// Geometry (the measured best for 1 x 2048 x 16384).
constexpr int kStripCols = 64;                              // columns per thread block
constexpr int kBoxRows = 128;                               // k rows per stage
constexpr int kStageBytes = kBoxRows * kStripCols * 2;      // 16 KiB
constexpr int kStages = 5;
constexpr int kConsumerWarps = 8;
constexpr int kConsumers = 32 * kConsumerWarps;
constexpr int kThreads = 32 + kConsumers;
constexpr int kMaxSliceBytes = 32 * 1024;                   // bf16 rows of A staged per block
constexpr int max_slice_k(int m_tile) { return kMaxSliceBytes / (2 * m_tile); }
constexpr int kMaxClusterK = 8;                             // k slices added inside one cluster
constexpr int kPrefetchBoxes = 6;                           // boxes asked into L2 before the wait
constexpr int kLanesPerRow = kStripCols / 8;                // 16-byte chunks per box row
constexpr int kRowsPerWarp = 32 / kLanesPerRow;             // box rows one warp-wide load covers
constexpr int kRowsPerPass = kRowsPerWarp * kConsumerWarps;
constexpr int kPasses = kBoxRows / kRowsPerPass;

struct StreamParams {
  const uint16_t* A;
  float* C;
  float* partial;
  int64_t a_batch, c_batch;       // batch strides in elements
  int64_t k, n;
  int64_t partial_split_stride;   // b * m * n
  int m;
  int strips;
  int split_k;
  int k_per_split;                // multiple of kBoxRows
  int overwrite;                  // 1: C = sum instead of C += sum
  int cluster_k;                  // 1: the k slices of a strip form a thread-block cluster and are
                                  //    added through distributed shared memory (no scratch)
  int a_bulk;                     // rows of A can be brought by bulk copies (16-byte alignment)
  uint32_t* status;
};

struct StreamBarriers {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t a_full;              // the bulk copies of the rows of A
  int abort_flag;
};

__device__ __forceinline__ void consumer_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Two f32 lanes in one 64-bit register, and acc = a * b + acc on both lanes at once
// (fma.rn.f32x2: each lane is an ordinary round-to-nearest FMA, so results equal two fmaf).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(uint64_t& acc, uint64_t a, uint64_t b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

template <int M_T, bool kClusterK>
__global__ void __launch_bounds__(kThreads)
gemv_stream_kernel(const __grid_constant__ CUtensorMap map_b, const StreamParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* ring = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  uint16_t* a_s = reinterpret_cast<uint16_t*>(ring + kStages * kStageBytes);  // [M_T][k_per_split] bf16
  float* red = reinterpret_cast<float*>(a_s + (size_t)p.k_per_split * M_T);   // [warp][M_T][64]
  float* out_s = red + kConsumerWarps * M_T * kStripCols;                     // [M_T][64]: this block's sums
  StreamBarriers* bars = reinterpret_cast<StreamBarriers*>(out_s + M_T * kStripCols);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // Cluster form: the split_k blocks of a strip are consecutive (they are one cluster and the
  // slice is the block's rank in it); otherwise slices are the slow index.
  const int strip = kClusterK ? blockIdx.x / p.split_k : blockIdx.x % p.strips;
  const int slice = kClusterK ? blockIdx.x % p.split_k : blockIdx.x / p.strips;
  const int bb = blockIdx.y;
  const int k0 = slice * p.k_per_split;
  const int k1 = (int)min((int64_t)k0 + p.k_per_split, p.k);
  const int boxes = (k1 - k0 + kBoxRows - 1) / kBoxRows;
  const int col0 = strip * kStripCols;
  const uint16_t* a_base = p.A + (int64_t)bb * p.a_batch + k0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], kConsumerWarps);
    }
    mbar_init(&bars->a_full, 1);
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_b);
    const int ahead = min(boxes, kPrefetchBoxes);
    for (int j = 0; j < ahead; ++j) tma_prefetch_l2_3d(&map_b, col0, k0 + j * kBoxRows, bb);
  } else if (warp == 1) {
    // The lines of A this block will stage (m rows of k1 - k0 bf16).
    const int lines = ((k1 - k0) * 2 + 127) / 128;
    for (int i = 0; i < p.m; ++i)
      for (int q = lane; q < lines; q += 32)
        prefetch_l2(reinterpret_cast<const uint8_t*>(a_base + (int64_t)i * p.k) + (size_t)q * 128);
  }
  __syncthreads();

  // Nothing above read or wrote global memory; from here on the preceding kernel on the
  // stream has completed and its writes are visible.
  pdl_wait();

  if (warp == 0) {
    // ---------------------------------------------------------------- producer
    if (elect_one()) {
      if (p.a_bulk) {
        // Row i of the slice of A: one bulk copy of (k1 - k0) bf16 (a multiple of 16 bytes
        // from a 16-byte-aligned address, which a_bulk asserts).
        const uint32_t row_bytes = (uint32_t)(k1 - k0) * 2u;
        mbar_arrive_expect_tx(&bars->a_full, row_bytes * (uint32_t)p.m);
        for (int i = 0; i < p.m; ++i)
          bulk_load(a_s + (size_t)i * p.k_per_split, a_base + (int64_t)i * p.k, row_bytes, &bars->a_full);
      }
      int stage = 0;
      uint32_t phase = 0;
      for (int j = 0; j < boxes; ++j) {
        if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag, p.status, 5)) break;
        mbar_arrive_expect_tx(&bars->full[stage], kStageBytes);
        tma_load_3d(ring + stage * kStageBytes, &map_b, &bars->full[stage], col0,
                    k0 + j * kBoxRows, bb);
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      // Every load of this block is in flight: the next kernel's blocks may come in.
      pdl_release();
    }
    return;
  }

  // ------------------------------------------------------------------- consumers
  const int ct = threadIdx.x - 32;          // 0 .. kConsumers - 1
  const int cw = warp - 1;
  const int chunk = lane % kLanesPerRow;    // columns [8 chunk, 8 chunk + 8) of the strip
  const int rg = lane / kLanesPerRow;       // row within the warp's group of rows

  // A[0:m, k0:k1) sits in shared memory as bf16, row i at a_s + i * k_per_split: brought by
  // the producer's bulk copies when alignment allows, else staged here.  B is zero past k
  // (TMA fill), so what A holds there does not matter as long as it is finite: zero it.
  const int staged = boxes * kBoxRows;
  if (!p.a_bulk) {
    for (int i = 0; i < p.m; ++i)
      for (int q = ct; q < k1 - k0; q += kConsumers)
        a_s[(size_t)i * p.k_per_split + q] = a_base[(int64_t)i * p.k + q];
  }
  for (int i = 0; i < M_T; ++i)
    for (int q = (i < p.m ? k1 - k0 : 0) + ct; q < staged; q += kConsumers)
      a_s[(size_t)i * p.k_per_split + q] = 0;
  // C is read now, long before it is needed, and added once at the very end.
  constexpr int kOutPerThread = (M_T * kStripCols + kConsumers - 1) / kConsumers;
  float c_in[kOutPerThread];
#pragma unroll
  for (int r = 0; r < kOutPerThread; ++r) {
    const int o = ct + r * kConsumers;
    const int i = o / kStripCols;
    const int64_t col = col0 + (o % kStripCols);
    c_in[r] = 0.f;
    if ((p.split_k == 1 || (kClusterK && slice == 0)) && !p.overwrite && o < M_T * kStripCols &&
        i < p.m && col < p.n)
      c_in[r] = p.C[(int64_t)bb * p.c_batch + (int64_t)i * p.n + col];
  }
  consumer_sync();

  uint64_t acc2[M_T][4];                  // columns (2h, 2h + 1) of the chunk, as f32 pairs
#pragma unroll
  for (int i = 0; i < M_T; ++i)
#pragma unroll
    for (int h = 0; h < 4; ++h) acc2[i][h] = 0ull;

  bool ok = true;
  if (p.a_bulk) {
    ok = mbar_wait(&bars->a_full, 0, abort_flag, p.status, 7);
    ok = __all_sync(0xffffffffu, ok);
  }
  {
    int stage = 0;
    uint32_t phase = 0;
    // Row (cw * kRowsPerWarp + rg + kRowsPerPass u) of a box, u = 0 .. kPasses - 1: 16 bytes
    // at column chunk `chunk`.
    const int row_in_box = cw * kRowsPerWarp + rg;
    const uint32_t lane_off = (uint32_t)(row_in_box * (kStripCols * 2) + chunk * 16);
    for (int j = 0; j < boxes && ok; ++j) {
      ok = mbar_wait(&bars->full[stage], phase, abort_flag, p.status, 6);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const uint8_t* src = ring + stage * kStageBytes + lane_off;
      uint4 v[kPasses];
#pragma unroll
      for (int u = 0; u < kPasses; ++u)
        v[u] = *reinterpret_cast<const uint4*>(src + u * kRowsPerPass * (kStripCols * 2));
      const uint16_t* a_col = a_s + j * kBoxRows + row_in_box;
#pragma unroll
      for (int u = 0; u < kPasses; ++u) {
        uint64_t a2[M_T];                 // the row's multiplier on both lanes
#pragma unroll
        for (int i = 0; i < M_T; ++i) {
          const float a = __uint_as_float(((uint32_t)a_col[(size_t)i * p.k_per_split + u * kRowsPerPass]) << 16);
          a2[i] = pack2(a, a);
        }
        const uint32_t ww[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const uint64_t b2 = pack2(bf16_lo(ww[h]), bf16_hi(ww[h]));
#pragma unroll
          for (int i = 0; i < M_T; ++i) fma2(acc2[i][h], a2[i], b2);
        }
      }
      __syncwarp();                       // every lane's reads of the stage are done
      if (lane == 0) mbar_arrive(&bars->empty[stage]);
      if (++stage == kStages) { stage = 0; phase ^= 1; }
    }
  }

  float acc[M_T][8];
#pragma unroll
  for (int i = 0; i < M_T; ++i)
#pragma unroll
    for (int h = 0; h < 4; ++h) unpack2(acc2[i][h], acc[i][2 * h], acc[i][2 * h + 1]);
  // Row groups of the warp, pairwise, in the same order in every lane.
#pragma unroll
  for (int i = 0; i < M_T; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float v = acc[i][j];
#pragma unroll
      for (int off = kLanesPerRow; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      acc[i][j] = v;
    }
  if (rg == 0) {
#pragma unroll
    for (int i = 0; i < M_T; ++i) {
      float4* dst = reinterpret_cast<float4*>(red + ((size_t)cw * M_T + i) * kStripCols + chunk * 8);
      dst[0] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      dst[1] = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
    }
  }
  consumer_sync();                        // reached by every consumer, timed out or not
  if (!kClusterK && *abort_flag) return;
  float sums[kOutPerThread];
#pragma unroll
  for (int r = 0; r < kOutPerThread; ++r) {
    const int o = ct + r * kConsumers;
    sums[r] = 0.f;
    if (o >= M_T * kStripCols) continue;
    const int i = o / kStripCols;
    float sum = red[(size_t)i * kStripCols + (o % kStripCols)];
#pragma unroll
    for (int w = 1; w < kConsumerWarps; ++w)
      sum += red[((size_t)w * M_T + i) * kStripCols + (o % kStripCols)];
    sums[r] = sum;
    if constexpr (kClusterK) out_s[o] = sum;
  }
  if constexpr (kClusterK) {
    // Every block of the cluster has parked its sums; block 0 adds them in slice order
    // (its own first), adds C once and stores.  The second barrier keeps the other blocks'
    // shared memory alive until block 0 has read it.  Both barriers are reached by every
    // consumer of every block, timed out or not (the producer warps have exited and do not
    // count), so no block can be left waiting.
    cluster_sync();
    if (slice == 0 && !*abort_flag) {
#pragma unroll
      for (int r = 0; r < kOutPerThread; ++r) {
        const int o = ct + r * kConsumers;
        const int i = o / kStripCols;
        const int64_t col = col0 + (o % kStripCols);
        if (o >= M_T * kStripCols || i >= p.m || col >= p.n) continue;
        float sum = sums[r];
        for (int s2 = 1; s2 < p.split_k; ++s2) sum += *peer_shared(out_s + o, (uint32_t)s2);
        p.C[(int64_t)bb * p.c_batch + (int64_t)i * p.n + col] = c_in[r] + sum;
      }
    }
    cluster_sync();
  } else {
#pragma unroll
    for (int r = 0; r < kOutPerThread; ++r) {
      const int o = ct + r * kConsumers;
      const int i = o / kStripCols;
      const int64_t col = col0 + (o % kStripCols);
      if (o >= M_T * kStripCols || i >= p.m || col >= p.n) continue;
      if (p.split_k == 1)
        p.C[(int64_t)bb * p.c_batch + (int64_t)i * p.n + col] = c_in[r] + sums[r];
      else
        p.partial[(int64_t)slice * p.partial_split_stride + ((int64_t)bb * p.m + i) * p.n + col] = sums[r];
    }
  }
}

// Tensor maps of B are cached per (pointer, shape).
struct BKey {
  const void* b;
  int64_t bsz, k, n;
  bool operator==(const BKey& o) const { return b == o.b && bsz == o.bsz && k == o.k && n == o.n; }
};
struct BEntry {
  BKey key;
  CUtensorMap map;
  uint64_t stamp;
  bool valid;
};
constexpr int kMapCache = 64;
BEntry g_bmaps[kMapCache];
uint64_t g_bstamp = 0;
std::mutex g_bmutex;

cudaError_t get_b_map(const BKey& key, CUtensorMap* out) {
  std::lock_guard<std::mutex> lock(g_bmutex);
  int victim = 0;
  for (int i = 0; i < kMapCache; ++i) {
    if (g_bmaps[i].valid && g_bmaps[i].key == key) {
      g_bmaps[i].stamp = ++g_bstamp;
      *out = g_bmaps[i].map;
      return cudaSuccess;
    }
    const uint64_t age_i = g_bmaps[i].valid ? g_bmaps[i].stamp : 0;
    const uint64_t age_v = g_bmaps[victim].valid ? g_bmaps[victim].stamp : 0;
    if (age_i < age_v) victim = i;
  }
  BEntry e{};
  e.key = key;
  // Promotion never reaches past the box row: a neighbouring strip's bytes belong to
  // another thread block.
  cudaError_t err = make_tensor_map_3d(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.b,
                                       (uint64_t)key.n, (uint64_t)key.k, (uint64_t)key.bsz,
                                       kStripCols, kBoxRows, CU_TENSOR_MAP_SWIZZLE_NONE,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
  if (err != cudaSuccess) return err;
  e.stamp = ++g_bstamp;
  e.valid = true;
  g_bmaps[victim] = e;
  *out = e.map;
  return cudaSuccess;
}

size_t smem_for(int m_tile, int k_per_split) {
  return 128 + (size_t)kStages * kStageBytes + (size_t)k_per_split * m_tile * 2 +
         (size_t)(kConsumerWarps + 1) * m_tile * kStripCols * 4 + sizeof(StreamBarriers) + 16;
}

template <int M_T, bool kClusterK>
cudaError_t launch(const StreamPlan& plan, const CUtensorMap& map, const StreamParams& prm,
                   int64_t b, cudaStream_t stream) {
  auto kern = gemv_stream_kernel<M_T, kClusterK>;
  static PerDeviceOnce once;   // the attribute belongs to the current device's copy of the kernel
  const cudaError_t attr_err = once.run_current([&] {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)smem_for(M_T, max_slice_k(M_T)));
  });
  if (attr_err != cudaSuccess) return attr_err;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(plan.strips * plan.split_k), (unsigned)b, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  int num_attrs = 1;
  if (plan.cluster_k) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)plan.split_k;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    num_attrs = 2;
  }
  cfg.attrs = attr;
  cfg.numAttrs = num_attrs;
  return cudaLaunchKernelEx(&cfg, kern, map, prm);
}

}  // namespace

bool stream_shape_supported(int64_t b, int m, int64_t k, int64_t n, const void* B) {
  if (b <= 0 || m <= 0 || m > 4 || k <= 0 || n <= 0) return false;
  if (n % 8 || reinterpret_cast<uintptr_t>(B) % 16) return false;   // TMA row pitch and base
  if (n >= (1ll << 31) || k >= (1ll << 31) || b >= (1ll << 31)) return false;
  return true;
}

// `split_k` 0: by shape.  `scratch_reduce`: keep the slices' sums in scratch and add them with
// the reduce kernel even where a cluster could (for tests and comparisons).
StreamPlan stream_plan(int sms, int64_t b, int m, int64_t k, int64_t n, int split_k, bool scratch_reduce) {
  StreamPlan pl{};
  pl.m_tile = m <= 1 ? 1 : m <= 2 ? 2 : 4;
  pl.strips = (int)((n + kStripCols - 1) / kStripCols);
  const int64_t blocks = b * pl.strips;
  const int slice_cap = max_slice_k(pl.m_tile);
  const int64_t max_s = (k + kBoxRows - 1) / kBoxRows;           // at least one box per slice
  const int64_t min_s = (k + slice_cap - 1) / slice_cap;         // the staged part of A must fit
  int64_t s = split_k;
  if (s <= 0) {
    // Two blocks per SM keep enough loads in flight; more slices only add reduce work.  The
    // planner's own choice is a power of two up to 8, so that the slices of a strip form a
    // cluster (the portable size limit) and pack the GPCs without leftovers.
    s = 1;
    if (blocks * 10 < (int64_t)sms * 13) {
      const int64_t want = std::min<int64_t>((2 * sms + blocks - 1) / blocks, k / 512);
      while (s * 2 <= want && s * 2 <= kMaxClusterK) s *= 2;
    }
    while (s < min_s && s < kMaxClusterK) s *= 2;
  }
  s = std::max<int64_t>(s, min_s);
  s = std::max<int64_t>(1, std::min<int64_t>(s, max_s));
  int64_t kps = (k + s - 1) / s;
  kps = (kps + kBoxRows - 1) / kBoxRows * kBoxRows;
  pl.k_per_split = (int)kps;
  pl.split_k = (int)((k + kps - 1) / kps);
  pl.supported = kps <= slice_cap;
  // Up to 8 slices are added inside a cluster; more (a forced split, or a k too long for 8
  // slices) go through scratch and the reduce kernel.
  pl.cluster_k = !scratch_reduce && pl.split_k > 1 && pl.split_k <= kMaxClusterK;
  pl.smem_bytes = smem_for(pl.m_tile, pl.k_per_split);
  pl.workspace_bytes = (pl.split_k > 1 && !pl.cluster_k) ? (size_t)pl.split_k * b * m * n * 4 : 0;
  return pl;
}

cudaError_t stream_launch(const DeviceInfo& dev, const StreamPlan& plan, int64_t b, int m, int64_t k,
                          int64_t n, const uint16_t* A, int64_t a_batch, const uint16_t* B, float* C,
                          int64_t c_batch, float* workspace, cudaStream_t stream,
                          uint64_t* launches, bool overwrite) {
  StreamParams prm{};
  prm.overwrite = overwrite ? 1 : 0;
  prm.a_batch = a_batch; prm.c_batch = c_batch;
  prm.k = k; prm.n = n;
  prm.partial_split_stride = b * m * n;
  prm.m = m;
  prm.strips = plan.strips;
  prm.split_k = plan.split_k;
  prm.cluster_k = plan.cluster_k ? 1 : 0;
  prm.k_per_split = plan.k_per_split;
  prm.a_bulk = (k % 8 == 0 && reinterpret_cast<uintptr_t>(A) % 16 == 0 && a_batch % 8 == 0) ? 1 : 0;
  prm.status = dev.status;
  // grid.y carries the batch index; larger batches go in slabs, each with its own map.
  for (int64_t b0 = 0; b0 < b; b0 += 65535) {
    const int64_t bn = std::min<int64_t>(65535, b - b0);
    CUtensorMap map;
    cudaError_t e = get_b_map(BKey{B + b0 * k * n, bn, k, n}, &map);
    if (e != cudaSuccess) return e;
    prm.A = A + b0 * a_batch;
    prm.C = C + b0 * c_batch;
    prm.partial = workspace ? workspace + b0 * m * n : nullptr;
    switch (plan.m_tile * 2 + (plan.cluster_k ? 1 : 0)) {
      case 2: e = launch<1, false>(plan, map, prm, bn, stream); break;
      case 3: e = launch<1, true>(plan, map, prm, bn, stream); break;
      case 4: e = launch<2, false>(plan, map, prm, bn, stream); break;
      case 5: e = launch<2, true>(plan, map, prm, bn, stream); break;
      case 8: e = launch<4, false>(plan, map, prm, bn, stream); break;
      default: e = launch<4, true>(plan, map, prm, bn, stream); break;
    }
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  if (plan.split_k > 1 && !plan.cluster_k) {
    cudaError_t e = skinny_reduce_launch(workspace, C, b, m, n, c_batch, plan.split_k, stream, overwrite);
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaSuccess;
}

}  // namespace morello
