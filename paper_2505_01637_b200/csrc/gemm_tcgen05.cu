// Tensor-core MatmulAccum for sm_100a: C[b] += A[b] x B[b] with bf16 operands and
// f32 accumulation in tensor memory.
//
// One persistent thread block per SM walks 128 x 256 output tiles.  Its warps are
// specialised:
//   warp 0   producer: TMA loads of a 128 x 64 tile of A and a 64 x 256 tile of B per
//            k block into a ring of shared-memory stages (128-byte swizzle);
//   warp 1   MMA issuer: one elected lane issues tcgen05.mma (M 128, N 256, K 16), four
//            per k block, accumulating in one of two 256-column TMEM buffers, and
//            commits to the stage's "empty" barrier and, after the last k block, to the
//            buffer's "full" barrier;
//   warps 2-5 epilogue: read the accumulator with tcgen05.ld (each warp its own 32-lane
//            quarter), add it to C in global memory (one rounding per element), and hand
//            the buffer back.  The epilogue of tile i overlaps the main loop of tile i+1.
// A is [m][k] (K-major operand).  B is [k][n], i.e. N is contiguous: it is fed as an
// MN-major operand, each 64-column group of the tile being one TMA box of 64 k rows.
// Rows, columns and k blocks past the tensor edge are zero-filled by TMA and the
// epilogue predicates its accesses, so m, n and k need not be multiples of the tile.
// Every barrier wait is bounded (sm100::mbar_wait); on a timeout the block stops
// issuing work, records a status word and exits after releasing its TMEM.
#include <algorithm>
#include <mutex>

#include "internal.h"
#include "sm100.cuh"
#include "tensormap.h"

namespace morello {
namespace {

using namespace sm100;

constexpr int kRowsPerCta = 128;                   // accumulator rows (TMEM lanes) per CTA
constexpr int kTileN = 256;                        // accumulator columns per tile
constexpr int kTileK = 64;                         // one 128-byte swizzle span of bf16
constexpr int kBytesA = kRowsPerCta * kTileK * 2;  // 16 KiB
constexpr int kBoxBytesB = kTileK * 64 * 2;        // one TMA box of B: 64 k rows x 64 columns
constexpr int kAccColumns = kTileN;                // f32 columns per accumulator buffer
constexpr int kTmemColumns = 2 * kAccColumns;      // 512: the whole tensor memory
constexpr int kThreads = 192;
constexpr int kMaxStages = 6;

// kPair = false: one CTA per 128 x 256 tile (cta_group::1), B tile whole in its
// shared memory.  kPair = true: two CTAs of a cluster share a 256 x 256 tile
// (cta_group::2): CTA r holds rows [128 r, 128 r + 128) of A and columns
// [128 r, 128 r + 128) of B, the leader (r = 0) issues the MMAs for both, and each
// CTA's epilogue drains its own 128 rows.  Halving B per CTA halves both the TMA fill
// and the operand reads of shared memory per MMA, which is what bounds the 1-CTA form.
template <bool kPair>
struct Shape {
  static constexpr int kCtas = kPair ? 2 : 1;
  static constexpr int kTileM = kRowsPerCta * kCtas;
  static constexpr int kColsB = kTileN / kCtas;          // columns of B held per CTA
  static constexpr int kBoxesB = kColsB / 64;
  static constexpr int kBytesB = kTileK * kColsB * 2;
  static constexpr int kStageBytes = kBytesA + kBytesB;  // 48 KiB / 32 KiB
  static constexpr int kStages = kPair ? 6 : 4;
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 /*alignment slack*/ + 256;
};

struct GemmParams {
  float* C;
  int64_t m, n, k;
  int64_t c_batch;  // m * n
  int m_tiles, n_tiles;
  int64_t tiles;    // b * m_tiles * n_tiles
  int k_blocks;
  uint32_t* status;
};

struct Barriers {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

template <bool kPair>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const GemmParams p) {
  using S = Shape<kPair>;
  extern __shared__ uint8_t smem_raw[];
  // Stage buffers must sit on 1024-byte boundaries (the swizzle pattern repeats every
  // 8 rows of 128 bytes and is keyed on address bits 7-9).  The carve-up is identical in
  // both CTAs of a pair: the pair MMA addresses the peer's operands by the same offsets.
  uint8_t* stages = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Barriers* bars = reinterpret_cast<Barriers*>(stages + (size_t)S::kStages * S::kStageBytes);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;  // 0 = leader of the pair
  const int64_t unit = kPair ? (blockIdx.x >> 1) : blockIdx.x;
  const int64_t units = kPair ? (gridDim.x >> 1) : gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&bars->full[s], S::kCtas);   // one arrive.expect_tx per producer of the pair
      mbar_init(&bars->empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->acc_full[i], 1);
      mbar_init(&bars->acc_empty[i], 4 * S::kCtas);  // one arrival per epilogue warp
    }
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_a);
    tma_prefetch_descriptor(&map_b);
  }
  if (warp == 1) {
    if constexpr (kPair) {
      tmem_alloc_pair(&bars->tmem_base, kTmemColumns);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(&bars->tmem_base, kTmemColumns);
      tmem_relinquish();
    }
  }
  tc_fence_before_sync();
  if constexpr (kPair) cluster_sync(); else __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  // Everything above touched no global memory; from here on the predecessor on the
  // stream must have completed.
  pdl_wait();
  pdl_release();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int64_t t = unit; t < p.tiles && ok; t += units) {
        const int mt = (int)(t % p.m_tiles);
        const int nt = (int)((t / p.m_tiles) % p.n_tiles);
        const int bb = (int)(t / ((int64_t)p.m_tiles * p.n_tiles));
        const int row0 = mt * S::kTileM + (int)rank * kRowsPerCta;
        const int col0 = nt * kTileN + (int)rank * S::kColsB;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!(ok = mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag, p.status, 1))) break;
          uint8_t* sa = stages + (size_t)stage * S::kStageBytes;
          uint8_t* sb = sa + kBytesA;
          if constexpr (kPair) {
            // Both producers report to the leader's barrier: it opens once both halves landed.
            const uint32_t full = map_to_cta(smem_u32(&bars->full[stage]), 0);
            mbar_arrive_expect_tx_cluster(full, S::kStageBytes);
            tma_load_3d_pair(sa, &map_a, full, kb * kTileK, row0, bb);
#pragma unroll
            for (int j = 0; j < S::kBoxesB; ++j)
              tma_load_3d_pair(sb + j * kBoxBytesB, &map_b, full, col0 + j * 64, kb * kTileK, bb);
          } else {
            mbar_arrive_expect_tx(&bars->full[stage], S::kStageBytes);
            tma_load_3d(sa, &map_a, &bars->full[stage], kb * kTileK, row0, bb);
#pragma unroll
            for (int j = 0; j < S::kBoxesB; ++j)
              tma_load_3d(sb + j * kBoxBytesB, &map_b, &bars->full[stage], col0 + j * 64,
                          kb * kTileK, bb);
          }
          if (++stage == S::kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = instr_desc_bf16(S::kTileM, kTileN, false, true);
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int64_t t = unit; t < p.tiles && ok; t += units) {
        if (!(ok = mbar_wait(&bars->acc_empty[buf], acc_phase ^ 1, abort_flag, p.status, 2))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * kAccColumns;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!(ok = mbar_wait(&bars->full[stage], phase, abort_flag, p.status, 3))) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(stages + (size_t)stage * S::kStageBytes);
          const uint32_t sb = sa + kBytesA;
#pragma unroll
          for (int j = 0; j < kTileK / 16; ++j) {
            // A, K-major: 8-row groups 1024 bytes apart; 16 k elements = 32 bytes along the row.
            const uint64_t da = smem_desc_sw128(sa + j * 32, 16, 1024);
            // B, MN-major: 64-column groups one TMA box (8 KiB) apart, 8-row k groups 1024 bytes
            // apart; 16 k rows = 2048 bytes.
            const uint64_t db = smem_desc_sw128(sb + j * 2048, kBoxBytesB, 1024);
            if constexpr (kPair) mma_bf16_ss_pair(d_tmem, da, db, idesc, (kb | j) != 0 ? 1u : 0u);
            else mma_bf16_ss(d_tmem, da, db, idesc, (kb | j) != 0 ? 1u : 0u);
          }
          // The stage is reusable (in both CTAs) once these MMAs have read it.
          if constexpr (kPair) mma_commit_pair(&bars->empty[stage], 3);
          else mma_commit(&bars->empty[stage]);
          if (++stage == S::kStages) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if constexpr (kPair) mma_commit_pair(&bars->acc_full[buf], 3);
        else mma_commit(&bars->acc_full[buf]);
        if (++buf == 2) { buf = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32 * quarter, 32 * quarter + 32)
    int buf = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int64_t t = unit; t < p.tiles && ok; t += units) {
      const int mt = (int)(t % p.m_tiles);
      const int nt = (int)((t / p.m_tiles) % p.n_tiles);
      const int64_t bb = t / ((int64_t)p.m_tiles * p.n_tiles);
      ok = mbar_wait(&bars->acc_full[buf], acc_phase, abort_flag, p.status, 4);
      ok = __all_sync(0xffffffffu, ok);  // also reconverges the warp for the aligned TMEM loads
      if (!ok) break;
      tc_fence_after_sync();
      const int64_t row = (int64_t)mt * S::kTileM + (int64_t)rank * kRowsPerCta + quarter * 32 + lane;
      const int64_t col0 = (int64_t)nt * kTileN;
      float* crow = p.C + bb * p.c_batch + row * p.n + col0;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * kAccColumns;
#pragma unroll 1
      for (int c = 0; c < kTileN; c += 64) {
        uint32_t r0[32], r1[32];
        tmem_ld_32x32(taddr + c, r0);
        tmem_ld_32x32(taddr + c + 32, r1);
        tmem_ld_wait();
        if (c + 64 == kTileN) {
          // The accumulator is in registers: hand the buffer back before the global traffic.
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if constexpr (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[buf]), 0));
            else mbar_arrive(&bars->acc_empty[buf]);
          }
        }
        if (row < p.m) {
          // C += acc: one reduction per element per call, performed at L2 (n % 4 == 0 here).
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            if (col0 + c + j < p.n)
              red_add_v4(crow + c + j, __uint_as_float(r0[j]), __uint_as_float(r0[j + 1]),
                         __uint_as_float(r0[j + 2]), __uint_as_float(r0[j + 3]));
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            if (col0 + c + 32 + j < p.n)
              red_add_v4(crow + c + 32 + j, __uint_as_float(r1[j]), __uint_as_float(r1[j + 1]),
                         __uint_as_float(r1[j + 2]), __uint_as_float(r1[j + 3]));
        }
      }
      if (++buf == 2) { buf = 0; acc_phase ^= 1; }
    }
  }

  __syncwarp();  // the elected lanes rejoin their warps before the aligned barriers below

  // Teardown: every role of both CTAs is done (or has given up) before shared and tensor
  // memory go away -- the pair MMA reads the peer's shared memory and the peer's epilogue
  // arrives on the leader's barriers.
  tc_fence_before_sync();
  if constexpr (kPair) cluster_sync(); else __syncthreads();
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    if constexpr (kPair) tmem_dealloc_pair(tmem_base, kTmemColumns);
    else tmem_dealloc(tmem_base, kTmemColumns);
  }
}

// Tensor maps are cached per (pointer, shape): encoding one costs a few microseconds.
struct MapKey {
  const void* a;
  const void* b;
  int64_t bsz, m, k, n;
  bool operator==(const MapKey& o) const {
    return a == o.a && b == o.b && bsz == o.bsz && m == o.m && k == o.k && n == o.n;
  }
};
struct MapEntry {
  MapKey key;
  CUtensorMap map_a, map_b;
  uint64_t stamp;
  bool valid;
};
constexpr int kMapCache = 32;
MapEntry g_maps[kMapCache];
uint64_t g_stamp = 0;
std::mutex g_map_mutex;

cudaError_t get_maps(const MapKey& key, CUtensorMap* ma, CUtensorMap* mb) {
  std::lock_guard<std::mutex> lock(g_map_mutex);
  int victim = 0;   // an unused slot if there is one, else the least recently used
  for (int i = 0; i < kMapCache; ++i) {
    if (g_maps[i].valid && g_maps[i].key == key) {
      g_maps[i].stamp = ++g_stamp;
      *ma = g_maps[i].map_a;
      *mb = g_maps[i].map_b;
      return cudaSuccess;
    }
    const uint64_t age_i = g_maps[i].valid ? g_maps[i].stamp : 0;
    const uint64_t age_v = g_maps[victim].valid ? g_maps[victim].stamp : 0;
    if (age_i < age_v) victim = i;
  }
  MapEntry e{};
  e.key = key;
  cudaError_t err = make_tensor_map_3d(&e.map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.a,
                                       (uint64_t)key.k, (uint64_t)key.m, (uint64_t)key.bsz, kTileK,
                                       kRowsPerCta, CU_TENSOR_MAP_SWIZZLE_128B);
  if (err != cudaSuccess) return err;
  err = make_tensor_map_3d(&e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.b, (uint64_t)key.n,
                           (uint64_t)key.k, (uint64_t)key.bsz, 64, kTileK,
                           CU_TENSOR_MAP_SWIZZLE_128B);
  if (err != cudaSuccess) return err;
  e.stamp = ++g_stamp;
  e.valid = true;
  g_maps[victim] = e;
  *ma = e.map_a;
  *mb = e.map_b;
  return cudaSuccess;
}

}  // namespace

bool gemm_shape_supported(int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                          const void* B, const void* C) {
  if (b <= 0 || m <= 0 || k <= 0 || n <= 0) return false;
  if (k % 8 || n % 8) return false;  // TMA row pitches must be multiples of 16 bytes
  if (reinterpret_cast<uintptr_t>(A) % 16 || reinterpret_cast<uintptr_t>(B) % 16 ||
      reinterpret_cast<uintptr_t>(C) % 16)
    return false;
  // Tensor-map extents are 32-bit, tile coordinates are ints.
  if (m >= (1ll << 31) || n >= (1ll << 31) || k >= (1ll << 31) || b >= (1ll << 31)) return false;
  return true;
}

// split_k is reused here as an experiment knob of the forced entry point: 1 forces the
// one-CTA form, 2 the pair form, 0 picks by shape.  No scratch is needed either way.
GemmPlan gemm_plan(int, int64_t, int64_t m, int64_t, int64_t, int split_k) {
  const bool pair = split_k == 2 || (split_k == 0 && m > kRowsPerCta);
  return GemmPlan{true, pair ? 2 : 1, 0};
}

namespace {

template <bool kPair>
cudaError_t launch_gemm(const DeviceInfo& dev, int64_t b, int64_t m, int64_t k, int64_t n,
                        const CUtensorMap& map_a, const CUtensorMap& map_b, float* C,
                        cudaStream_t stream) {
  using S = Shape<kPair>;
  static std::once_flag once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(once, [] {
    attr_err = cudaFuncSetAttribute(gemm_kernel<kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)S::kSmemBytes);
  });
  if (attr_err != cudaSuccess) return attr_err;

  GemmParams p{};
  p.C = C;
  p.m = m; p.n = n; p.k = k;
  p.c_batch = m * n;
  p.m_tiles = (int)((m + S::kTileM - 1) / S::kTileM);
  p.n_tiles = (int)((n + kTileN - 1) / kTileN);
  p.tiles = b * p.m_tiles * (int64_t)p.n_tiles;
  p.k_blocks = (int)((k + kTileK - 1) / kTileK);
  p.status = dev.status;

  const int64_t max_units = kPair ? dev.sms / 2 : dev.sms;
  const int64_t units = std::min<int64_t>(p.tiles, max_units);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(units * S::kCtas), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = S::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  int num_attrs = 1;
  if (kPair) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    num_attrs = 2;
  }
  cfg.attrs = attr;
  cfg.numAttrs = num_attrs;
  return cudaLaunchKernelEx(&cfg, gemm_kernel<kPair>, map_a, map_b, p);
}

}  // namespace

cudaError_t gemm_launch(const DeviceInfo& dev, const GemmPlan& plan, int64_t b, int64_t m, int64_t k,
                        int64_t n, const uint16_t* A, const uint16_t* B, float* C, float*,
                        cudaStream_t stream, uint64_t* launches) {
  CUtensorMap map_a, map_b;
  cudaError_t e = get_maps(MapKey{A, B, b, m, k, n}, &map_a, &map_b);
  if (e != cudaSuccess) return e;
  e = plan.split_k == 2 ? launch_gemm<true>(dev, b, m, k, n, map_a, map_b, C, stream)
                        : launch_gemm<false>(dev, b, m, k, n, map_a, map_b, C, stream);
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace morello
