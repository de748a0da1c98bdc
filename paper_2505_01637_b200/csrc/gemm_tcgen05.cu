// Tensor-core MatmulAccum for sm_100a: C[b] += A[b] x B[b] with bf16 operands and
// f32 accumulation in tensor memory.
//
// Persistent thread blocks (one per SM) walk output tiles.  Two forms:
//   one CTA per tile   (cta_group::1): tile 128 x N, N in {64, 128, 256};
//   a CTA pair per tile (cta_group::2): tile 256 x N, N in {128, 256}; CTA r of the
//       pair holds rows [128 r, 128 r + 128) of A and columns [N/2 r, N/2 r + N/2) of B,
//       the leader (r = 0) issues the MMAs for both, each CTA drains its own 128 rows.
// Warps are specialised:
//   warp 0   producer: TMA loads of a 128 x 64 tile of A and a 64 x (N or N/2) tile of B
//            per k block into a ring of shared-memory stages (128-byte swizzle);
//   warp 1   MMA issuer: one elected lane issues tcgen05.mma (K 16), four per k block,
//            accumulating in one of two TMEM buffers, and commits to the stage's "empty"
//            barrier and, after the last k block, to the buffer's "full" barrier;
//   warps 2-5 epilogue: read the accumulator with tcgen05.ld (each warp its own 32-lane
//            quarter) 32 columns at a time, park the 32 x 32 block in shared memory in
//            the 128-byte-swizzled layout and hand it to the TMA engine as a reduce-add
//            into C (cp.reduce.async.bulk.tensor ... add.f32): one addition per element,
//            performed in L2, nothing read back by the SM.  The epilogue of tile i
//            overlaps the main loop of tile i+1.
// A is [m][k] (K-major operand).  B is [k][n], i.e. N is contiguous: it is fed as an
// MN-major operand, each 64-column group of the tile being one TMA box of 64 k rows.
// Rows, columns and k blocks past the tensor edge are zero-filled by the TMA loads and
// clipped by the TMA reduce, so m, n and k need not be multiples of the tile.
// When the rows of C are not addressable by the TMA engine (a row pitch that is not a multiple
// of 16 bytes, or a base that is not 16-byte aligned: the padded-copy route) the epilogue warps
// add their sums to C straight from registers instead, one L2 reduction (or store) per element.
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
constexpr int kTileK = 64;                         // one 128-byte swizzle span of bf16
constexpr int kBytesA = kRowsPerCta * kTileK * 2;  // 16 KiB
constexpr int kBoxBytesB = kTileK * 64 * 2;        // one TMA box of B: 64 k rows x 64 columns
constexpr int kAccStride = 256;                    // TMEM columns between the two accumulators
constexpr int kTmemColumns = 2 * kAccStride;       // 512: the whole tensor memory
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;
constexpr int kEpiCols = 32;                       // columns per epilogue block (128 bytes of f32)
constexpr int kEpiBlockBytes = 32 * kEpiCols * 4;  // one warp's 32 x 32 block
constexpr int kEpiBytes = 4 * 2 * kEpiBlockBytes;  // 4 warps x 2 blocks in flight
constexpr int kSmemBudget = 227 * 1024;

template <bool kPair, int kTileN>
struct Shape {
  static constexpr int kCtas = kPair ? 2 : 1;
  static constexpr int kTileM = kRowsPerCta * kCtas;
  static constexpr int kColsB = kTileN / kCtas;          // columns of B held per CTA
  static constexpr int kBoxesB = kColsB / 64;
  static constexpr int kBytesB = kTileK * kColsB * 2;
  static constexpr int kStageBytes = kBytesA + kBytesB;
  static constexpr int kFit = (kSmemBudget - kEpiBytes - 1024 - 256) / kStageBytes;
  static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
  static constexpr size_t kSmemBytes =
      (size_t)kStages * kStageBytes + kEpiBytes + 1024 /*alignment slack*/ + 256;
  static_assert(kColsB % 64 == 0 && kTileN <= kAccStride, "tile shape");
};

// Height of the TMA box of A: a whole 128-row tile, or, when the matrix has fewer rows than
// that (then there is one row of tiles, in the one-CTA form), m rounded up to a multiple of 16.
inline int a_box_rows(int64_t m) {
  return m >= kRowsPerCta ? kRowsPerCta : (int)((m + 15) / 16 * 16);
}

struct GemmParams {
  float* C;
  int64_t m, n, k;
  int64_t c_batch;  // m * n
  int m_tiles, n_tiles;
  int64_t tiles;    // b * m_tiles * n_tiles
  int64_t whole;    // work items [0, whole) are whole tiles, in tile order;
  int64_t items;    // items [whole, items) are the column halves of tiles [whole, tiles)
  int raster_g;     // rows of tiles per group of the tile order (see decode_item); 0: all of them
  int k_blocks;
  int ws_split;     // > 1: few tiles and a long k -- every tile's k range is cut into this many
                    // slices, each an item of its own whose sums go (as a plain store) to
                    // partial[slice][b][m][n]; the slice-ordered reduce kernel adds them and C
  int kb_per_slice; // k blocks per slice
  int64_t bsz;      // batches
  int seg_blocks;   // > 0: k blocks per segment of the k range (see KSegments); 0: k as stored
  uint32_t seg_a, seg_b;
  int pack_strip;   // > 0: B is packed in strips of this many columns (a multiple of 64)
  int pack_strips;  // strips per batch
  uint32_t* status;
  int overwrite;   // 1: C = product (TMA store) instead of C += product (TMA reduce-add)
  int bt;          // 1: B is stored column-major, [b][n][k]: the K-major operand (boxes of 64 k x 64 columns)
  int a_box_rows;  // rows of A one TMA box brings: 128, or m rounded up to 16 when m < 128
  int c_direct;    // 1: C is written from registers (its rows have c_cols columns, c_cols <= n,
  int64_t c_cols;  //    and need no alignment beyond 4 bytes); the tensor map of C is not used
};

struct Barriers {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};

// One unit of work of a thread block (or pair): a tile, or the left / right column half of one.
// First stored k element of k block kb of the call: kb * 64, or, with segments, block kb's
// place inside the stored term its segment reads.
__device__ __forceinline__ int k_coord(int kb, int seg_blocks, uint32_t terms) {
  if (seg_blocks == 0) return kb * kTileK;
  const int s = kb / seg_blocks;
  return ((int)((terms >> (3 * s)) & 7u) * seg_blocks + (kb - s * seg_blocks)) * kTileK;
}

// TMA coordinates of the 64-column box of B at (first column `col`, first k element `kc`) of
// batch bb: row-major B is {n, k, b}; column-major {k, n, b}; packed in strips of `strip`
// columns {strip, k, b * strips} (the strip index folded into the batch coordinate).
struct BBox { int x, y, z; };
__device__ __forceinline__ BBox b_box(int bt, int strip, int strips, int col, int kc, int bb) {
  if (bt) return BBox{kc, col, bb};
  if (strip) {
    const int st = col / strip;
    return BBox{col - st * strip, kc, bb * strips + st};
  }
  return BBox{col, kc, bb};
}
// The same box at another k: only the k coordinate changes (the strip arithmetic, a division,
// is done once per item, outside the k loop).
__device__ __forceinline__ BBox at_k(BBox box, int bt, int kc) {
  if (bt) box.x = kc; else box.y = kc;
  return box;
}

struct Item {
  int mt, nt, bb;
  int n_off;   // first column of the item inside its tile
  int cols;    // columns of the item: the tile's width or half of it
  int kb0, kb1;  // k blocks [kb0, kb1) of the item
  int out_b;   // batch coordinate of the item's output in the map the epilogue stores through
};
template <int kTileN>
__device__ __forceinline__ Item decode_item(const GemmParams& p, int64_t t) {
  Item it;
  int64_t tile = t;
  it.n_off = 0;
  it.cols = kTileN;
  it.kb0 = 0;
  it.kb1 = p.k_blocks;
  int slice = 0;
  if (p.ws_split > 1) {            // items are (tile, slice); no halves in this mode
    tile = t / p.ws_split;
    slice = (int)(t - tile * p.ws_split);
    it.kb0 = slice * p.kb_per_slice;
    it.kb1 = min(p.k_blocks, it.kb0 + p.kb_per_slice);
  } else if (t >= p.whole) {
    const int64_t h = t - p.whole;
    tile = p.whole + (h >> 1);
    it.cols = kTileN / 2;
    it.n_off = (int)(h & 1) * (kTileN / 2);
  }
  // Tiles are numbered group by group: a group is raster_g rows of tiles (all of them when 0),
  // walked row-fastest and then column by column, so that the tiles in flight at any time share
  // a few rows of A and a few columns of B (both then stay in L2 while the wave passes).
  // Batches are outermost.
  const int64_t per_batch = (int64_t)p.m_tiles * p.n_tiles;
  it.bb = (int)(tile / per_batch);
  const int within = (int)(tile - it.bb * per_batch);
  if (p.raster_g > 0) {
    const int per_group = p.raster_g * p.n_tiles;
    const int grp = within / per_group, r = within - grp * per_group;
    const int rows = min(p.raster_g, p.m_tiles - grp * p.raster_g);
    it.nt = r / rows;
    it.mt = grp * p.raster_g + (r - it.nt * rows);
  } else {
    it.nt = within / p.m_tiles;
    it.mt = within - it.nt * p.m_tiles;
  }
  it.out_b = (int)(slice * p.bsz + it.bb);
  return it;
}

template <bool kPair, int kTileN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_c, const GemmParams p) {
  using S = Shape<kPair, kTileN>;
  extern __shared__ uint8_t smem_raw[];
  // Stage buffers must sit on 1024-byte boundaries (the swizzle pattern repeats every
  // 8 rows of 128 bytes and is keyed on address bits 7-9).  The carve-up is identical in
  // both CTAs of a pair: the pair MMA addresses the peer's operands by the same offsets.
  uint8_t* stages = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* epi = stages + (size_t)S::kStages * S::kStageBytes;   // 1024-byte aligned as well
  Barriers* bars = reinterpret_cast<Barriers*>(epi + kEpiBytes);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = kPair ? cluster_ctarank() : 0u;  // 0 = leader of the pair
  const int64_t unit = kPair ? (blockIdx.x >> 1) : blockIdx.x;
  const int64_t units = kPair ? (gridDim.x >> 1) : gridDim.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&bars->full[s], 1);          // the (leader's) producer's arrive.expect_tx
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
    if (!p.c_direct) tma_prefetch_descriptor(&map_c);
  }
  if (p.a_box_rows < kRowsPerCta) {
    // Few rows: the TMA box of A is only as high as m needs (a box that is mostly outside the
    // tensor loads several times slower than its in-bounds part alone).  The rows of the stage
    // the box never writes are zeroed once, here; the MMA reads them as zeros.
    for (int s2 = 0; s2 < S::kStages; ++s2) {
      uint4* z = reinterpret_cast<uint4*>(stages + (size_t)s2 * S::kStageBytes);
      for (int q = threadIdx.x; q < kBytesA / 16; q += kThreads) z[q] = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async_smem();
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
      const uint32_t leader_full = kPair ? map_to_cta(smem_u32(&bars->full[0]), 0) : 0u;
      (void)leader_full;
      for (int64_t t = unit; t < p.items && ok; t += units) {
        const Item it = decode_item<kTileN>(p, t);
        const int bb = it.bb;
        const int row0 = it.mt * S::kTileM + (int)rank * kRowsPerCta;
        const int cols_b = it.cols / S::kCtas;            // columns of B this CTA brings
        const int boxes_b = cols_b / 64;
        const int col0 = it.nt * kTileN + it.n_off + (int)rank * cols_b;
        const uint32_t stage_tx = (uint32_t)(boxes_b * kBoxBytesB + p.a_box_rows * (kTileK * 2));
        BBox boxes[S::kBoxesB];
#pragma unroll
        for (int j = 0; j < S::kBoxesB; ++j)
          boxes[j] = b_box(p.bt, p.pack_strip, p.pack_strips, col0 + j * 64, 0, bb);
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
          if (!(ok = mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag, p.status, 1))) break;
          uint8_t* sa = stages + (size_t)stage * S::kStageBytes;
          uint8_t* sb = sa + kBytesA;
          const int ka = k_coord(kb, p.seg_blocks, p.seg_a), kbb = k_coord(kb, p.seg_blocks, p.seg_b);
          if constexpr (kPair) {
            // Both CTAs' loads complete on the leader's barrier.  Only the leader arrives on
            // it (a local arrive, announcing the bytes of both halves): a load of the peer
            // that lands first just leaves the byte count negative until then, and the phase
            // cannot end before the leader's arrival.
            const uint32_t full = leader_full + (uint32_t)stage * 8u;
            if (rank == 0)
              mbar_arrive_expect_tx(&bars->full[stage], 2 * stage_tx);
            tma_load_3d_pair(sa, &map_a, full, ka, row0, bb);
#pragma unroll
            for (int j = 0; j < S::kBoxesB; ++j)
              if (j < boxes_b) {
                const BBox c = at_k(boxes[j], p.bt, kbb);
                tma_load_3d_pair(sb + j * kBoxBytesB, &map_b, full, c.x, c.y, c.z);
              }
          } else {
            mbar_arrive_expect_tx(&bars->full[stage], stage_tx);
            tma_load_3d(sa, &map_a, &bars->full[stage], ka, row0, bb);
#pragma unroll
            for (int j = 0; j < S::kBoxesB; ++j)
              if (j < boxes_b) {
                const BBox c = at_k(boxes[j], p.bt, kbb);
                tma_load_3d(sb + j * kBoxBytesB, &map_b, &bars->full[stage], c.x, c.y, c.z);
              }
          }
          if (++stage == S::kStages) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (rank == 0 && elect_one()) {
      // B row-major is the MN-major operand, B column-major the K-major one.
      const uint32_t idesc_tile = p.bt ? instr_desc_bf16(S::kTileM, kTileN, false, false)
                                       : instr_desc_bf16(S::kTileM, kTileN, false, true);
      const uint32_t idesc_half = p.bt ? instr_desc_bf16(S::kTileM, kTileN / 2, false, false)
                                       : instr_desc_bf16(S::kTileM, kTileN / 2, false, true);
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int64_t t = unit; t < p.items && ok; t += units) {
        const Item it = decode_item<kTileN>(p, t);
        const uint32_t idesc = it.cols == kTileN ? idesc_tile : idesc_half;
        if (!(ok = mbar_wait(&bars->acc_empty[buf], acc_phase ^ 1, abort_flag, p.status, 2))) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * kAccStride;
        for (int kb = it.kb0; kb < it.kb1; ++kb) {
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
            // (K-major B: like A -- its 64-row boxes follow each other, 8-row groups 1024 bytes
            // apart, 32 bytes per K step.)
            const uint64_t db = p.bt ? smem_desc_sw128(sb + j * 32, 16, 1024)
                                     : smem_desc_sw128(sb + j * 2048, kBoxBytesB, 1024);
            const uint32_t accumulate = ((kb - it.kb0) | j) != 0 ? 1u : 0u;
            if constexpr (kPair) mma_bf16_ss_pair(d_tmem, da, db, idesc, accumulate);
            else mma_bf16_ss(d_tmem, da, db, idesc, accumulate);
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
    uint8_t* my_blocks = epi + (size_t)quarter * 2 * kEpiBlockBytes;
    // Row `lane` of a block is 128 bytes; its 16-byte chunk j sits at chunk j ^ (lane % 8)
    // (the 128-byte swizzle the tensor map of C expects), which also spreads a quarter
    // warp's stores over all banks.
    const uint32_t row_off = (uint32_t)lane * 128u;
    const uint32_t sw = (uint32_t)(lane & 7);
    int buf = 0;
    uint32_t acc_phase = 0;
    uint32_t blk = 0;              // alternates between this warp's two blocks
    bool ok = true;
    for (int64_t t = unit; t < p.items && ok; t += units) {
      const Item it = decode_item<kTileN>(p, t);
      const int mt = it.mt;
      ok = mbar_wait(&bars->acc_full[buf], acc_phase, abort_flag, p.status, 4);
      ok = __all_sync(0xffffffffu, ok);  // also reconverges the warp for the aligned TMEM loads
      if (!ok) break;
      tc_fence_after_sync();
      const int row0 = mt * S::kTileM + (int)rank * kRowsPerCta + quarter * 32;
      const int col0 = it.nt * kTileN + it.n_off;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * kAccStride;
      const bool rows_live = row0 < p.m;   // warp-uniform
      if (p.c_direct) {
        // Straight from registers.  The 16-lane load shape hands every thread pairs of
        // neighbouring columns of four rows, so that one warp-wide access covers 8 rows x 32
        // contiguous bytes; every element goes out as one L2 reduction (or one store).
        float* c_base = p.C + (int64_t)it.out_b * p.c_batch;
        const int r_lo = row0 + (lane >> 2);            // this thread's rows: r_lo + 0, 8, 16, 24
        const int c_lo = col0 + 2 * (lane & 3);
#pragma unroll 1
        for (int c = 0; c < it.cols; c += 64) {
          uint32_t r0[32], r1[32];
          tmem_ld_16x64(taddr + c, r0);                          // lanes 0-15 of the quarter
          tmem_ld_16x64(taddr + ((uint32_t)16 << 16) + c, r1);   // lanes 16-31
          tmem_ld_wait();
          if (c + 64 >= it.cols) {
            // The accumulator has left tensor memory: hand the buffer back to the MMA issuer.
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
              if constexpr (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[buf]), 0));
              else mbar_arrive(&bars->acc_empty[buf]);
            }
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const int row = r_lo + 8 * h;
              if (row >= p.m) continue;
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int col = c_lo + c + 8 * q + e;
                if (col >= p.c_cols) continue;
                float* dst = c_base + (int64_t)row * p.c_cols + col;
                const uint32_t v = (h < 2 ? r0 : r1)[4 * q + 2 * (h & 1) + e];
                if (p.overwrite) *dst = __uint_as_float(v); else red_add_f32(dst, v);
              }
            }
          }
        }
        if (++buf == 2) { buf = 0; acc_phase ^= 1; }
        continue;
      }
#pragma unroll 1
      for (int c = 0; c < it.cols; c += kEpiCols) {
        const bool live = rows_live && (col0 + c < p.n);
        uint32_t r[32];
        if (live) {
          // The block written two steps ago must have been read by the TMA engine.
          if (lane == 0) bulk_wait_group_read<1>();
          __syncwarp();
          tmem_ld_32x32(taddr + c, r);
          tmem_ld_wait();
        }
        if (c + kEpiCols == it.cols) {
          // The accumulator has left tensor memory: hand the buffer back to the MMA issuer.
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            if constexpr (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[buf]), 0));
            else mbar_arrive(&bars->acc_empty[buf]);
          }
        }
        if (live) {
          const uint32_t dst = smem_u32(my_blocks + blk * kEpiBlockBytes) + row_off;
#pragma unroll
          for (int j = 0; j < 8; ++j)
            st_shared_v4(dst + (((uint32_t)j ^ sw) << 4), r[4 * j], r[4 * j + 1], r[4 * j + 2],
                         r[4 * j + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            // C[bb, row0 : row0 + 32, col0 + c : col0 + c + 32] += block; rows and columns
            // past the edge of C are dropped by the TMA engine.
            if (p.overwrite) tma_store_3d(&map_c, my_blocks + blk * kEpiBlockBytes, col0 + c, row0, it.out_b);
            else tma_reduce_add_3d(&map_c, my_blocks + blk * kEpiBlockBytes, col0 + c, row0, it.out_b);
            bulk_commit_group();
          }
          blk ^= 1u;
        }
      }
      if (++buf == 2) { buf = 0; acc_phase ^= 1; }
    }
    // Shared memory must outlive the engine's reads, and the additions must have been
    // performed before the kernel counts as complete.
    if (lane == 0) bulk_wait_group<0>();
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

// ---------------------------------------------------------------------------------------
// Few rows (m <= 64): the operands trade places.  C^T[n, m] += B^T[n, k] x A^T[k, m]: a thread
// block owns a strip of 128 columns of B, which becomes the M side of the MMA (B is [k][n], so
// it is the MN-major operand here too: two TMA boxes of 64 k rows x 64 columns per k block,
// the same boxes the tiles above use), and the rows of A, rounded up to a multiple of 16,
// are its N side (K-major, one box of 64 k x kRowsA rows per k block).  The MMA's cost then
// follows m instead of a fixed 128 rows, the accumulator is 128 lanes x kRowsA columns, and
// the epilogue holds one column of C per thread: for every row i a warp adds 32 consecutive
// floats of C (C is read before the main loop, the sum is added once, at the end).
// The call streams B once and is bound by HBM.  Up to 16 rows the block is kept small enough
// (108 KiB of stages, 32 TMEM columns) for the next call's block to be resident beside it:
// before its griddepcontrol.wait that block asks the TMA engine to prefetch its first k
// blocks of B into L2 (nothing reaches the SM, so this is legal early), and a block lets
// dependents launch once its producer has issued its last load.  With more rows a stage
// carries more of A and the same budget would hold too little of B in flight: the ring then
// takes 200 KiB and the next call's block follows when this one leaves.
constexpr int kSwapRingKiB = 108;        // stages of the <= 16-row kernel: two blocks fit an SM
constexpr int kSwapBigRingKiB = 200;     // stages with more rows of A
template <int kRowsA>
struct SwapShape {
  static constexpr int kBytesStrip = 2 * kBoxBytesB;                  // 128 columns x 64 k: 16 KiB
  static constexpr int kBytesRows = kRowsA * kTileK * 2;              // 2 .. 8 KiB
  static constexpr int kStageBytes = kBytesStrip + kBytesRows;
  static constexpr int kRingKiB = kRowsA <= 16 ? kSwapRingKiB : kSwapBigRingKiB;
  static constexpr int kFit = (kRingKiB * 1024) / kStageBytes;
  static constexpr int kStages = kFit < kMaxStages ? kFit : kMaxStages;
  static constexpr int kTmemCols = kRowsA <= 32 ? 32 : 64;
  static constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + 1024 /*alignment slack*/ + 256;
  static_assert(kRowsA % 16 == 0 && kRowsA >= 16 && kRowsA <= 64, "rows of A");
};
constexpr int kSwapStripCols = 128;
constexpr int kSwapMaxRows = 64;
constexpr int kSwapPrefetchBlocks = 6;   // k blocks asked into L2 before the wait

struct SwapParams {
  float* C;
  int bt;           // 1: B is stored column-major, [b][n][k]
  int overwrite;    // 1: C = product instead of C += product
  int64_t m, n;
  int64_t c_batch;  // m * c_cols
  int64_t c_cols;   // columns (and row pitch) of C: n, or fewer when B was padded with zero columns
  int k_blocks;
  int split_k;      // k slices per strip (cluster form: the slices of a strip are one cluster;
                    // otherwise every slice writes its own copy of the output, see the kernel)
  int kb_per_slice; // k blocks per slice
  int strips;       // 128-column strips per batch
  int64_t items;    // batches x strips x slices
  int64_t bsz;      // batches
  int seg_blocks;   // > 0: k blocks per segment of the k range (see KSegments); 0: k as stored
  uint32_t seg_a, seg_b;
  int pack_strip;   // > 0: B is packed in strips of this many columns (a multiple of 64)
  int pack_strips;  // strips per batch
  uint32_t* status;
};

struct SwapBarriers {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t acc_full;
  uint64_t acc_empty;
  uint32_t tmem_base;
  int abort_flag;
};

// kClusterK: few strips and a long k -- the k range is cut into 2, 4 or 8 slices, the blocks
// of a strip form a thread-block cluster, each parks its accumulator in its own shared memory
// (the stage ring is free by then) and the blocks share the rows out among themselves: each adds
// its rows' slices through distributed shared memory in slice order, then C: one launch, no
// scratch, a fixed order.
// Without a cluster the grid is persistent: a block walks the (batch, strip, slice) items
// blockIdx.x, blockIdx.x + gridDim.x, ...; its producer keeps the stage ring full across items,
// so the loads of the next items run under the epilogue of the current one.  With many short
// items (batched problems with a short k) that removes the per-block set-up from the critical
// path.  With one item per block (the long streams the kernel was tuned on) nothing changes.
template <int kRowsA, bool kClusterK, bool kPersistent>
__global__ void __launch_bounds__(kThreads)
swap_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const SwapParams p) {
  using S = SwapShape<kRowsA>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* stages = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  SwapBarriers* bars = reinterpret_cast<SwapBarriers*>(stages + (size_t)S::kStages * S::kStageBytes);
  volatile int* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  static_assert(!(kClusterK && kPersistent), "a cluster takes one item per block");
  // Items: one per block (blockIdx.x = strip x slice, blockIdx.y = batch: the loops below then
  // run once and cost nothing), or, persistent, item t = (batch * strips + strip) * slices +
  // slice walked in strides of the grid.
  const int per_batch = p.strips * p.split_k;
  const int first = kPersistent ? (int)blockIdx.x : 0;
  const int stride = kPersistent ? (int)gridDim.x : 1;
  const int last = kPersistent ? (int)p.items : first + 1;     // items [first, last) in steps of stride
  struct Work { int bb, col0, slice, kb_begin, kb_end; };
  auto decode = [&](int t) {
    Work w;
    int r;
    if constexpr (kPersistent) {
      w.bb = t / per_batch;
      r = t - w.bb * per_batch;
    } else {
      w.bb = (int)blockIdx.y;
      r = (int)blockIdx.x;
    }
    w.col0 = (r / p.split_k) * kSwapStripCols;
    w.slice = r % p.split_k;
    w.kb_begin = w.slice * p.kb_per_slice;
    w.kb_end = min(p.k_blocks, w.kb_begin + p.kb_per_slice);
    return w;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < S::kStages; ++s) {
      mbar_init(&bars->full[s], 1);
      mbar_init(&bars->empty[s], 1);
    }
    mbar_init(&bars->acc_full, 1);
    mbar_init(&bars->acc_empty, 4);     // one arrival per epilogue warp
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_descriptor(&map_a);
    tma_prefetch_descriptor(&map_b);
    if (first < last) {
      const Work w = decode(first);
      const int ahead = min(w.kb_end, w.kb_begin + kSwapPrefetchBlocks);
      const BBox box0 = b_box(p.bt, p.pack_strip, p.pack_strips, w.col0, 0, w.bb);
      const BBox box1 = b_box(p.bt, p.pack_strip, p.pack_strips, w.col0 + 64, 0, w.bb);
      for (int kb = w.kb_begin; kb < ahead; ++kb) {
        const int kbb = k_coord(kb, p.seg_blocks, p.seg_b);
        const BBox c0 = at_k(box0, p.bt, kbb), c1 = at_k(box1, p.bt, kbb);
        tma_prefetch_l2_3d(&map_b, c0.x, c0.y, c0.z);
        tma_prefetch_l2_3d(&map_b, c1.x, c1.y, c1.z);
      }
    }
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, S::kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = bars->tmem_base;

  // Nothing above read or wrote global memory; from here on the predecessor on the stream has
  // completed.
  pdl_wait();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = first; t < last && ok; t += stride) {
        const Work w = decode(t);
        const BBox box0 = b_box(p.bt, p.pack_strip, p.pack_strips, w.col0, 0, w.bb);
        const BBox box1 = b_box(p.bt, p.pack_strip, p.pack_strips, w.col0 + 64, 0, w.bb);
        for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
          if (!(ok = mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag, p.status, 8))) break;
          uint8_t* sb = stages + (size_t)stage * S::kStageBytes;
          uint8_t* sa = sb + S::kBytesStrip;
          mbar_arrive_expect_tx(&bars->full[stage], S::kStageBytes);
          const int ka = k_coord(kb, p.seg_blocks, p.seg_a), kbb = k_coord(kb, p.seg_blocks, p.seg_b);
          const BBox c0 = at_k(box0, p.bt, kbb), c1 = at_k(box1, p.bt, kbb);
          tma_load_3d(sb, &map_b, &bars->full[stage], c0.x, c0.y, c0.z);
          tma_load_3d(sb + kBoxBytesB, &map_b, &bars->full[stage], c1.x, c1.y, c1.z);
          tma_load_3d(sa, &map_a, &bars->full[stage], ka, 0, w.bb);
          if (++stage == S::kStages) { stage = 0; phase ^= 1; }
        }
      }
      // Every load of this block is in flight: the next kernel's blocks may come in.
      pdl_release();
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (elect_one()) {
      // M = 128 columns of B (MN-major A operand), N = kRowsA rows of A (K-major B operand).
      // (With B column-major the strip is a K-major operand like the rows of A.)
      const uint32_t idesc = p.bt ? instr_desc_bf16(kSwapStripCols, kRowsA, false, false)
                                  : instr_desc_bf16(kSwapStripCols, kRowsA, true, false);
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = first; t < last && ok; t += stride) {
        const Work w = decode(t);
        // The epilogue has read the previous item's sums out of the accumulator.
        if constexpr (kPersistent) {
          if (!(ok = mbar_wait(&bars->acc_empty, acc_phase ^ 1, abort_flag, p.status, 11))) break;
          tc_fence_after_sync();
        }
        for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
          if (!(ok = mbar_wait(&bars->full[stage], phase, abort_flag, p.status, 9))) break;
          tc_fence_after_sync();
          const uint32_t sb = smem_u32(stages + (size_t)stage * S::kStageBytes);
          const uint32_t sa = sb + S::kBytesStrip;
#pragma unroll
          for (int j = 0; j < kTileK / 16; ++j) {
            // The strip of B: 64-column groups one TMA box apart, 8-row k groups 1024 bytes
            // apart, 16 k rows = 2048 bytes.  The rows of A: 8-row groups 1024 bytes apart,
            // 16 k elements = 32 bytes along the row.
            const uint64_t d_strip = p.bt ? smem_desc_sw128(sb + j * 32, 16, 1024)
                                          : smem_desc_sw128(sb + j * 2048, kBoxBytesB, 1024);
            const uint64_t d_rows = smem_desc_sw128(sa + j * 32, 16, 1024);
            mma_bf16_ss(tmem_base, d_strip, d_rows, idesc, ((kb - w.kb_begin) | j) != 0 ? 1u : 0u);
          }
          mma_commit(&bars->empty[stage]);
          if (++stage == S::kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) mma_commit(&bars->acc_full);
        acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32 * quarter, 32 * quarter + 32)
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int t = first; t < last; t += stride) {
      const Work w = decode(t);
      const int slice = w.slice;
      const int64_t col = (int64_t)w.col0 + quarter * 32 + lane;   // this thread's column of C
      const bool col_live = col < p.c_cols;
      // Without a cluster, slices > 1 means that C is partial[slice][b][m][n] in the workspace.
      const int64_t out_b = kClusterK ? w.bb : (int64_t)slice * p.bsz + w.bb;
      float* c_col = p.C + out_b * p.c_batch + col;
      // Cluster form: block r of the cluster finishes the rows i with i % split_k == r.
      float c_in[kRowsA];
#pragma unroll
      for (int i = 0; i < kRowsA; ++i) {
        const bool mine = !kClusterK || (i % p.split_k) == slice;
        c_in[i] = (mine && col_live && i < p.m && !p.overwrite) ? c_col[(int64_t)i * p.c_cols] : 0.f;
      }
      if (ok) ok = mbar_wait(&bars->acc_full, acc_phase, abort_flag, p.status, 10);
      ok = __all_sync(0xffffffffu, ok);  // also reconverges the warp for the aligned TMEM loads
      acc_phase ^= 1;
      if (ok) {
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        // Cluster form: every MMA has completed, so the stage ring is free; the accumulator is
        // parked there as part[row][128 columns of the strip].
        float* part = reinterpret_cast<float*>(stages);
#pragma unroll
        for (int g = 0; g < kRowsA / 16; ++g) {
          uint32_t r[16];
          tmem_ld_32x16(taddr + g * 16, r);
          tmem_ld_wait();
          if (kPersistent && g == kRowsA / 16 - 1) {
            // The last of the sums is in registers: the MMA warp may start the next item.
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty);
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            if constexpr (kClusterK) {
              part[(g * 16 + i) * kSwapStripCols + quarter * 32 + lane] = __uint_as_float(r[i]);
            } else {
              if (col_live && g * 16 + i < p.m)
                c_col[(int64_t)(g * 16 + i) * p.c_cols] = c_in[g * 16 + i] + __uint_as_float(r[i]);
            }
          }
        }
      } else if (!kClusterK) {
        break;      // timed out: nothing more is written (the cluster form still meets its barriers)
      }
      if constexpr (kClusterK) {
        // Both cluster barriers are executed by every thread of every block (see below); between
        // them every block finishes its share of the rows: the slices' sums in slice order (read
        // through distributed shared memory), then C, then the store.
        __syncwarp();
        cluster_sync();
        if (!*abort_flag) {
          const float* part = reinterpret_cast<const float*>(stages);
#pragma unroll
          for (int i = 0; i < kRowsA; ++i) {
            if (!col_live || i >= p.m || (i % p.split_k) != slice) continue;
            const float* mine = part + i * kSwapStripCols + quarter * 32 + lane;
            float sum = *peer_shared(mine, 0u);
            for (int s2 = 1; s2 < p.split_k; ++s2) sum += *peer_shared(mine, (uint32_t)s2);
            c_col[(int64_t)i * p.c_cols] = c_in[i] + sum;
          }
        }
        __syncwarp();
        cluster_sync();
      }
    }
  }
  if constexpr (kClusterK) {
    if (warp < 2) {        // producer and MMA warps take part in the two cluster barriers too
      __syncwarp();
      cluster_sync();
      cluster_sync();
    }
  }

  __syncwarp();
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem_base, S::kTmemCols);
  }
}

// Tensor maps are cached per (pointers, shape): encoding one costs a few microseconds.
struct MapKey {
  const void* a;
  const void* b;
  const void* c;
  int64_t bsz, m, k, n;
  int bt;    // layout of B: 0 row-major, 1 column-major, >= 64 packed in strips of that many columns
  int64_t c_bsz;   // batches of the output map: bsz, or slices x bsz when c is the workspace;
                   // 0: no map of C is wanted (the kernel writes C from registers)
  bool operator==(const MapKey& o) const {
    return a == o.a && b == o.b && c == o.c && bsz == o.bsz && m == o.m && k == o.k && n == o.n &&
           bt == o.bt && c_bsz == o.c_bsz;
  }
};
struct MapEntry {
  MapKey key;
  CUtensorMap map_a, map_b, map_c;
  uint64_t stamp;
  bool valid;
};
constexpr int kMapCache = 64;
MapEntry g_maps[kMapCache];
uint64_t g_stamp = 0;
std::mutex g_map_mutex;

cudaError_t get_maps(const MapKey& key, CUtensorMap* ma, CUtensorMap* mb, CUtensorMap* mc) {
  std::lock_guard<std::mutex> lock(g_map_mutex);
  int victim = 0;   // an unused slot if there is one, else the least recently used
  for (int i = 0; i < kMapCache; ++i) {
    if (g_maps[i].valid && g_maps[i].key == key) {
      g_maps[i].stamp = ++g_stamp;
      *ma = g_maps[i].map_a;
      *mb = g_maps[i].map_b;
      *mc = g_maps[i].map_c;
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
                                       (uint32_t)a_box_rows(key.m), CU_TENSOR_MAP_SWIZZLE_128B);
  if (err != cudaSuccess) return err;
  // Either way a box is 64 x 64 elements with 128-byte rows: [k][n] gives 64 k rows of 64
  // columns, [n][k] gives 64 columns (rows of the stored matrix) of 64 k.
  if (key.bt == 1)
    err = make_tensor_map_3d(&e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.b, (uint64_t)key.k,
                             (uint64_t)key.n, (uint64_t)key.bsz, kTileK, 64,
                             CU_TENSOR_MAP_SWIZZLE_128B);
  else if (key.bt >= 64)   // packed: {strip, k, b x strips}; a box is again 64 k rows of 64 columns
    err = make_tensor_map_3d(&e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.b, (uint64_t)key.bt,
                             (uint64_t)key.k, (uint64_t)(key.bsz * ((key.n + key.bt - 1) / key.bt)), 64,
                             kTileK, CU_TENSOR_MAP_SWIZZLE_128B);
  else
    err = make_tensor_map_3d(&e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, key.b, (uint64_t)key.n,
                             (uint64_t)key.k, (uint64_t)key.bsz, 64, kTileK,
                             CU_TENSOR_MAP_SWIZZLE_128B);
  if (err != cudaSuccess) return err;
  if (key.c_bsz > 0)
    err = make_tensor_map_3d(&e.map_c, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, key.c, (uint64_t)key.n,
                             (uint64_t)key.m, (uint64_t)key.c_bsz, kEpiCols, 32,
                             CU_TENSOR_MAP_SWIZZLE_128B);
  if (err != cudaSuccess) return err;
  e.stamp = ++g_stamp;
  e.valid = true;
  g_maps[victim] = e;
  *ma = e.map_a;
  *mb = e.map_b;
  *mc = e.map_c;
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

namespace {

template <bool kPair, int kTileN>
cudaError_t set_smem_attribute() {
  static PerDeviceOnce once;   // the attribute belongs to the current device's copy of the kernel
  return once.run_current([] {
    return cudaFuncSetAttribute(gemm_kernel<kPair, kTileN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Shape<kPair, kTileN>::kSmemBytes);
  });
}

// How many CTA pairs the device can hold at once.  A pair needs two SMs of one
// cluster-scheduling domain, so this can be fewer than sms / 2; a persistent grid larger
// than it would run its surplus pairs only after the first ones have finished.
constexpr int kMaxDevices = 64;
int g_pair_units[kMaxDevices];   // 0 = not asked yet
std::mutex g_pair_mutex;

int pair_units(int sms) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return std::max(1, sms / 2);
  std::lock_guard<std::mutex> lock(g_pair_mutex);
  if (g_pair_units[dev] > 0) return g_pair_units[dev];
  int clusters = 0;
  if (set_smem_attribute<true, 256>() == cudaSuccess) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(sms / 2 * 2), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = Shape<true, 256>::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&clusters, gemm_kernel<true, 256>, &cfg) != cudaSuccess) {
      (void)cudaGetLastError();
      clusters = 0;
    }
  }
  if (clusters <= 0) clusters = std::max(1, sms / 2 - 8);   // conservative when the query fails
  clusters = std::min(clusters, std::max(1, sms / 2));
  g_pair_units[dev] = clusters;
  return clusters;
}

}  // namespace

int gemm_pair_units(int sms) { return pair_units(sms); }

// The knob of the forced entry point (its split_k argument) selects the kernel and its tile:
// knob % 16 = form (0 by shape, 1 one CTA per tile, 2 a CTA pair per tile, 3 operand-swapped),
// (knob / 16) % 16 = tile columns / 64 (0 by shape; 1, 2 or 4; with form 3 the number of k slices
// inside a cluster), + 256 keeps the last wave's tiles whole, (knob / 512) % 16 = k slices through
// the workspace (0 by shape, 1 none, 2 .. 8).
//
// By shape: with a single row of tiles (m <= 128) the call streams B once and is bound by
// memory, so the widest tile that still gives about one thread block per SM wins.  Otherwise
// the candidate with the least "waves x k blocks x columns" wins, a wave being one tile per SM
// (or per pair), weighted by what the narrower and the one-CTA tiles were measured to cost per
// column (they re-read A more often, and a lone CTA reads the whole B tile from its own shared
// memory).
//
// Few tiles and a long k: a call whose tiles fill less than half the device is cut along k as
// well.  Each (tile, slice) item stores its sums to partial[slice][b][m][n] in the workspace
// and one more launch adds the slices in slice order, then C -- the bits do not depend on which
// block finished first.
namespace {

constexpr int kRasterRows = 8;                   // rows of tiles per group of the tile order
constexpr int kWsMaxSplit = 8;
constexpr int kWsMinBlocks = 16;                 // k blocks a slice keeps at least
constexpr size_t kWsMaxBytes = size_t(64) << 20; // partial sums stay well inside L2

// The largest number of k slices (<= want) whose partial sums fit the workspace cap and that
// leaves no slice empty.
int ws_fit(int want, int64_t k_blocks, int64_t b, int64_t m, int64_t n) {
  int split = std::max(1, std::min(want, kWsMaxSplit));
  while (split > 1 && (size_t)split * b * m * n * 4 > kWsMaxBytes) --split;
  while (split > 1 && (k_blocks + split - 1) / split * (split - 1) >= k_blocks) --split;
  return split;
}

}  // namespace

GemmPlan gemm_plan(int sms, int64_t b, int64_t m, int64_t k, int64_t n, int knob) {
  if (knob < 0) return GemmPlan{false, 0, 0, 0, false, 1, 1};
  const int forced_g = (knob / 8192) % 64;
  const int forced_ws = (knob / 512) % 16;
  const bool halves = ((knob / 256) % 2) == 0;
  knob %= 256;
  int form = knob % 16, tile_n = (knob / 16) * 64;
  const int64_t k_blocks = (k + kTileK - 1) / kTileK;
  if (forced_ws > kWsMaxSplit) return GemmPlan{false, 0, 0, 0, false, 1, 1};
  auto finish = [&](GemmPlan plan) {
    if (plan.ws_split > 1) {
      plan.workspace_bytes = (size_t)plan.ws_split * b * m * n * 4;
      plan.halves = false;
    }
    // The tile order: groups of kRasterRows rows of tiles unless the knob says otherwise (63: a
    // column of tiles at a time).
    plan.raster_g = forced_g == 63 ? 0 : forced_g != 0 ? forced_g : kRasterRows;
    return plan;
  };
  // By shape, the k slices of `tiles` items on `units` units.
  auto ws_by_shape = [&](int64_t tiles, int64_t units) {
    if (forced_ws != 0) return ws_fit(forced_ws, k_blocks, b, m, n);
    if (tiles * 2 > units || k_blocks < 2 * kWsMinBlocks) return 1;
    const int64_t want = std::min<int64_t>(units / tiles, k_blocks / kWsMinBlocks);
    return ws_fit((int)std::min<int64_t>(want, kWsMaxSplit), k_blocks, b, m, n);
  };
  // Form 3: the operand-swapped kernel.  By shape it takes every call of at most 64 rows.
  // Beyond 64 rows the 128-row tiles win: an accumulator of more than 64 columns per thread
  // cannot be paired with an early read of C in registers.
  if (form == 3 || (form == 0 && tile_n == 0 && m <= kSwapMaxRows)) {
    // With form 3 the knob's column field is the number of k slices instead (0 = by shape).
    const int forced_split = tile_n / 64;
    if (m > kSwapMaxRows || (b > 65535 && forced_split > 1) ||
        (forced_split != 0 && forced_split != 1 && forced_split != 2 && forced_split != 4 && forced_split != 8))
      return GemmPlan{false, 0, 0, 0, false, 1, 1};
    const int64_t strips = b * ((n + kSwapStripCols - 1) / kSwapStripCols);
    int split = forced_split;
    if (split == 0) {
      // Few strips and a long k: cut k inside a cluster.  That pays up to 16 rows and up to 32
      // strips (with more rows a block fills an SM and clusters of such blocks pack badly; with
      // more strips the device is busy anyway): as many slices as leave eight k blocks each.  The
      // other shapes of few strips go through the workspace.
      split = 1;
      if (forced_ws <= 1 && a_box_rows(m) == 16 && strips <= 32 && b <= 65535)
        while (split < 8 && k_blocks >= 8 * split) split *= 2;
    }
    while (split > 1 && (k_blocks + split - 1) / split * (split - 1) >= k_blocks) split /= 2;   // no empty slice
    int ws = 1;
    if (split == 1) ws = ws_by_shape(strips, sms);
    return finish(GemmPlan{true, 3, a_box_rows(m), 0, false, split, ws});
  }
  if (form < 0 || form > 2 || (tile_n != 0 && tile_n != 64 && tile_n != 128 && tile_n != 256) ||
      (form == 2 && tile_n == 64))
    return GemmPlan{false, 0, 0, 0, false, 1, 1};
  if (form != 2 && tile_n == 0 && m <= kRowsPerCta) {
    // First without k slices (they cost a second launch and a trip through the workspace); with
    // them only when even 64-column tiles leave the device idle.
    for (int tn = 256; tn >= 64; tn >>= 1) {
      const int64_t tiles = b * ((n + tn - 1) / tn);
      if (tiles * 5 >= (int64_t)sms * 4 && forced_ws <= 1) return finish(GemmPlan{true, 1, tn, 0, halves, 1, 1});
    }
    int best_n = 64;
    for (int tn = 256; tn >= 64; tn >>= 1) {
      const int64_t tiles = b * ((n + tn - 1) / tn);
      if (tiles * ws_by_shape(tiles, sms) * 5 >= (int64_t)sms * 4) { best_n = tn; break; }
    }
    const int64_t tiles = b * ((n + best_n - 1) / best_n);
    return finish(GemmPlan{true, 1, best_n, 0, halves, 1, ws_by_shape(tiles, sms)});
  }
  double best = 0;
  int best_form = 0, best_n = 0, best_ws = 1;
  for (int f = 1; f <= 2; ++f) {
    if (form != 0 && f != form) continue;
    if (form == 0 && f == 2 && m <= kRowsPerCta) continue;   // a pair would idle its second CTA
    for (int tn = 256; tn >= 64; tn >>= 1) {
      if ((tile_n != 0 && tn != tile_n) || (f == 2 && tn == 64)) continue;
      const int64_t tile_m = (int64_t)kRowsPerCta * f;
      const int64_t tiles = b * ((m + tile_m - 1) / tile_m) * ((n + tn - 1) / tn);
      const int64_t units = std::max(1, f == 2 ? pair_units(sms) : sms);
      const int ws = ws_by_shape(tiles, units);
      const int64_t items = tiles * ws;
      const int64_t tail = items % units;
      const bool cut = ws == 1 && halves && tiles > units && tail > 0 && 2 * tail <= units &&
                       (tn / f / 2) % 64 == 0;
      // A last wave cut into halves costs about 0.6 of a whole one.
      const double waves = (double)(items / units) + (tail == 0 ? 0.0 : cut ? 0.625 : 1.0);
      // In units of one column of one k block on a pair's 256-column tile (about 1.5 ns).  The
      // launch that adds the slices: about 3 us and its bytes at L2 speed.
      double cost = waves * (double)((k_blocks + ws - 1) / ws) * tn * (f == 1 ? 1.15 : 1.0) *
                    (tn == 256 ? 1.0 : tn == 128 ? 1.25 : 1.6);
      if (ws > 1) cost += 2000.0 + (double)(ws + 2) * b * m * n * 4 / 4.5e3;
      if (best_n == 0 || cost < best) { best = cost; best_form = f; best_n = tn; best_ws = ws; }
    }
  }
  if (best_n == 0) return GemmPlan{false, 0, 0, 0, false, 1, 1};
  return finish(GemmPlan{true, best_form, best_n, 0, halves, 1, best_ws});
}

namespace {

template <bool kPair, int kTileN>
cudaError_t launch_gemm(const DeviceInfo& dev, int64_t b, int64_t m, int64_t k, int64_t n,
                        const CUtensorMap& map_a, const CUtensorMap& map_b,
                        const CUtensorMap& map_c, float* C, bool halves, int ws_split, int raster_g,
                        int64_t c_cols, bool overwrite, int bt, const KSegments* seg, cudaStream_t stream) {
  using S = Shape<kPair, kTileN>;
  const cudaError_t attr_err = set_smem_attribute<kPair, kTileN>();
  if (attr_err != cudaSuccess) return attr_err;

  GemmParams p{};
  p.C = C;
  p.m = m; p.n = n; p.k = k;
  p.c_direct = c_cols > 0 ? 1 : 0;
  p.c_cols = c_cols > 0 ? c_cols : n;
  p.c_batch = m * p.c_cols;
  p.m_tiles = (int)((m + S::kTileM - 1) / S::kTileM);
  p.n_tiles = (int)((n + kTileN - 1) / kTileN);
  p.tiles = b * p.m_tiles * (int64_t)p.n_tiles;
  p.whole = p.tiles;
  p.items = p.tiles;
  p.k_blocks = (int)((k + kTileK - 1) / kTileK);
  p.status = dev.status;
  p.a_box_rows = a_box_rows(m);
  p.overwrite = overwrite ? 1 : 0;
  p.bt = bt == 1 ? 1 : 0;
  p.pack_strip = bt >= 64 ? bt : 0;
  p.pack_strips = bt >= 64 ? (int)((n + bt - 1) / bt) : 0;
  p.bsz = b;
  p.raster_g = raster_g > 0 && raster_g < p.m_tiles ? raster_g : 0;
  if (seg) { p.seg_blocks = seg->blocks; p.seg_a = seg->a_terms; p.seg_b = seg->b_terms; }
  p.ws_split = std::max(1, ws_split);
  p.kb_per_slice = (p.k_blocks + p.ws_split - 1) / p.ws_split;
  if (p.ws_split > 1) {      // map_c covers the partial sums; every item stores its own
    p.items = p.tiles * p.ws_split;
    p.whole = p.items;
    p.overwrite = 1;
    halves = false;
  }

  const int64_t max_units = kPair ? pair_units(dev.sms) : dev.sms;
  // The last wave of a compute-bound problem: when its tiles would occupy at most half the
  // units, each is cut into two column halves so that twice as many units share the wave.
  // (Its k is not cut: a second addition into C would make the bits depend on arrival order,
  // and a trip through the workspace costs more than it saves here.)
  const int64_t tail = p.tiles % max_units;
  if (halves && (S::kColsB / 2) % 64 == 0 && p.tiles > max_units && tail > 0 && 2 * tail <= max_units) {
    p.whole = p.tiles - tail;
    p.items = p.whole + 2 * tail;
  }
  const int64_t units = std::min<int64_t>(p.items, max_units);
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
  return cudaLaunchKernelEx(&cfg, gemm_kernel<kPair, kTileN>, map_a, map_b, map_c, p);
}

}  // namespace

namespace {

// Blocks of the operand-swapped kernel the device holds at once: two per SM with the small ring.
template <int kRowsA>
int64_t swap_resident(int sms) { return (int64_t)sms * (kRowsA <= 16 ? 2 : 1); }

template <int kRowsA, bool kClusterK, bool kPersistent>
cudaError_t launch_swap_form(const DeviceInfo& dev, int split, int64_t b, int64_t m, int64_t k, int64_t n,
                             const CUtensorMap& map_a, const CUtensorMap& map_b, float* C, int64_t c_cols,
                             bool overwrite, int bt, const KSegments* seg, cudaStream_t stream) {
  using S = SwapShape<kRowsA>;
  static PerDeviceOnce once;   // the attribute belongs to the current device's copy of the kernel
  const cudaError_t attr_err = once.run_current([] {
    return cudaFuncSetAttribute(swap_kernel<kRowsA, kClusterK, kPersistent>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)S::kSmemBytes);
  });
  if (attr_err != cudaSuccess) return attr_err;
  SwapParams p{};
  p.bt = bt == 1 ? 1 : 0;
  p.pack_strip = bt >= 64 ? bt : 0;
  p.pack_strips = bt >= 64 ? (int)((n + bt - 1) / bt) : 0;
  p.overwrite = overwrite ? 1 : 0;
  p.m = m; p.n = n;
  p.c_cols = c_cols > 0 ? c_cols : n;
  p.c_batch = m * p.c_cols;
  p.k_blocks = (int)((k + kTileK - 1) / kTileK);
  p.split_k = std::max(1, split);
  p.bsz = b;
  p.kb_per_slice = (p.k_blocks + p.split_k - 1) / p.split_k;
  p.status = dev.status;
  if (seg) { p.seg_blocks = seg->blocks; p.seg_a = seg->a_terms; p.seg_b = seg->b_terms; }
  const int64_t strips = (n + kSwapStripCols - 1) / kSwapStripCols;
  // Cluster form: grid.y carries the batch index (the planner keeps batches beyond a grid
  // dimension off this kernel).
  if ((!kPersistent && b > 65535) || strips * p.split_k >= (1ll << 31)) return cudaErrorInvalidValue;
  p.C = C;
  p.strips = (int)strips;
  p.items = b * strips * p.split_k;
  cudaLaunchConfig_t cfg{};
  if (!kPersistent) {
    cfg.gridDim = dim3((unsigned)(strips * p.split_k), (unsigned)b, 1);
  } else {
    // Persistent: the items shared out evenly among as many blocks as fit the device at once.
    if (p.items >= (1ll << 31)) return cudaErrorInvalidValue;
    const int64_t resident = swap_resident<kRowsA>(dev.sms);
    const int64_t per_block = (p.items + resident - 1) / resident;
    cfg.gridDim = dim3((unsigned)((p.items + per_block - 1) / per_block), 1, 1);
  }
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = S::kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  int num_attrs = 1;
  if (kClusterK) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.split_k;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    num_attrs = 2;
  }
  cfg.attrs = attr;
  cfg.numAttrs = num_attrs;
  return cudaLaunchKernelEx(&cfg, swap_kernel<kRowsA, kClusterK, kPersistent>, map_a, map_b, p);
}

// `split` > 1: the slices of a strip form a cluster and C is the output.  `ws_split` > 1: the
// slices are independent blocks and C is the workspace, partial[slice][b][m][n].
template <int kRowsA>
cudaError_t launch_swap(const DeviceInfo& dev, int split, int ws_split, int64_t b, int64_t m, int64_t k,
                        int64_t n, const CUtensorMap& map_a, const CUtensorMap& map_b, float* C,
                        int64_t c_cols, bool overwrite, int bt, const KSegments* seg, cudaStream_t stream) {
  if (split > 1)
    return launch_swap_form<kRowsA, true, false>(dev, split, b, m, k, n, map_a, map_b, C, c_cols, overwrite, bt,
                                                 seg, stream);
  // More items than blocks fit at once (and batches beyond a grid dimension): persistent.
  const int64_t items = b * ((n + kSwapStripCols - 1) / kSwapStripCols) * std::max(1, ws_split);
  if (items > swap_resident<kRowsA>(dev.sms) || b > 65535)
    return launch_swap_form<kRowsA, false, true>(dev, ws_split, b, m, k, n, map_a, map_b, C, c_cols, overwrite,
                                                 bt, seg, stream);
  return launch_swap_form<kRowsA, false, false>(dev, ws_split, b, m, k, n, map_a, map_b, C, c_cols, overwrite,
                                                bt, seg, stream);
}

}  // namespace

cudaError_t gemm_launch(const DeviceInfo& dev, const GemmPlan& plan, int64_t b, int64_t m, int64_t k,
                        int64_t n, const uint16_t* A, const uint16_t* B, float* C, float* workspace,
                        cudaStream_t stream, uint64_t* launches, bool overwrite, int bt,
                        const KSegments* seg, int64_t c_cols) {
  // With k slices through the workspace the kernels write partial[slice][b][m][n] there (plain
  // stores) and the reduce launch below adds the slices and C.
  const bool sliced = plan.ws_split > 1;
  if (sliced && !workspace) return cudaErrorInvalidValue;
  if (c_cols < 0 || c_cols > n) return cudaErrorInvalidValue;
  float* out = sliced ? workspace : C;
  const bool out_overwrite = sliced ? true : overwrite;
  // c_cols > 0: C is [b][m][c_cols], written from registers by the kernels (or, sliced, by the
  // reduce launch); the partial sums in the workspace keep the kernels' own n columns.
  const int64_t direct = sliced ? 0 : c_cols;
  CUtensorMap map_a, map_b, map_c;
  // With segments the stored operands are shorter along k than the call's k range.
  if (seg && (seg->blocks <= 0 || k % (64ll * seg->blocks) != 0 || k / (64ll * seg->blocks) > 8))
    return cudaErrorInvalidValue;
  cudaError_t e = get_maps(MapKey{A, B, out, b, m, seg ? seg->k_stored : k, n, bt,
                                  direct > 0 ? 0 : sliced ? plan.ws_split * b : b},
                           &map_a, &map_b, &map_c);
  if (e != cudaSuccess) return e;
  const int code = plan.form * 1000 + plan.tile_n;
  const int wss = plan.ws_split, rg = plan.raster_g;
  const bool hv = plan.halves;
  switch (code) {
    case 3016: e = launch_swap<16>(dev, plan.split_k, wss, b, m, k, n, map_a, map_b, out, direct, out_overwrite, bt, seg, stream); break;
    case 3032: e = launch_swap<32>(dev, plan.split_k, wss, b, m, k, n, map_a, map_b, out, direct, out_overwrite, bt, seg, stream); break;
    case 3048: e = launch_swap<48>(dev, plan.split_k, wss, b, m, k, n, map_a, map_b, out, direct, out_overwrite, bt, seg, stream); break;
    case 3064: e = launch_swap<64>(dev, plan.split_k, wss, b, m, k, n, map_a, map_b, out, direct, out_overwrite, bt, seg, stream); break;
    case 1064: e = launch_gemm<false, 64>(dev, b, m, k, n, map_a, map_b, map_c, out, hv, wss, rg, direct, out_overwrite, bt, seg, stream); break;
    case 1128: e = launch_gemm<false, 128>(dev, b, m, k, n, map_a, map_b, map_c, out, hv, wss, rg, direct, out_overwrite, bt, seg, stream); break;
    case 1256: e = launch_gemm<false, 256>(dev, b, m, k, n, map_a, map_b, map_c, out, hv, wss, rg, direct, out_overwrite, bt, seg, stream); break;
    case 2128: e = launch_gemm<true, 128>(dev, b, m, k, n, map_a, map_b, map_c, out, hv, wss, rg, direct, out_overwrite, bt, seg, stream); break;
    case 2256: e = launch_gemm<true, 256>(dev, b, m, k, n, map_a, map_b, map_c, out, hv, wss, rg, direct, out_overwrite, bt, seg, stream); break;
    default: return cudaErrorInvalidValue;
  }
  if (e != cudaSuccess) return e;
  ++*launches;
  if (sliced) {
    e = skinny_reduce_launch(workspace, C, b, (int)m, n, m * (c_cols > 0 ? c_cols : n), plan.ws_split, stream,
                             overwrite, c_cols);
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaSuccess;
}

}  // namespace morello
