// Internal declarations shared by the translation units of the CUDA library.
// `overwrite` selects the non-accumulating operation everywhere: C = A x B, C's prior contents
// neither read nor added.
// Nothing here is visible through the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <mutex>

namespace morello {

// Set-up that has to happen once per device and not once per process: a kernel's function
// attributes (the opt-in to more than 48 KiB of dynamic shared memory, say) belong to the
// current device's copy of the kernel.  run(dev, fn) calls fn() the first time it sees device
// `dev` and hands back its result; a failure is not remembered, the next call tries again.
// Devices beyond the table run fn() every time (a cheap host call).
class PerDeviceOnce {
 public:
  static constexpr int kSlots = 64;
  template <typename F>
  cudaError_t run(int dev, F&& fn) {
    if (dev < 0 || dev >= kSlots) return fn();
    std::lock_guard<std::mutex> lock(mutex_);
    if (done_[dev]) return cudaSuccess;
    const cudaError_t e = fn();
    done_[dev] = (e == cudaSuccess);
    return e;
  }
  // The same, for the device that is current on the calling thread.
  template <typename F>
  cudaError_t run_current(F&& fn) {
    int dev = -1;
    const cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    return run(dev, static_cast<F&&>(fn));
  }

 private:
  std::mutex mutex_;
  bool done_[kSlots] = {};
};

// Device-side status word written by bounded waits that gave up.
// 0 = OK; otherwise (site << 16) | detail, first writer wins.
struct DeviceInfo {
  int sms = 0;
  int cc_major = 0;
  uint32_t* status = nullptr;  // one zero-initialised word in device memory
};

// ---- skinny path (FP32 FMA, rows in chunks of <= 16) -------------------------
struct SkinnyPlan {
  int m_tile;        // 1, 2, 4, 8 or 16: compile-time row count of the kernel used
  int vec;           // bf16 elements per load: 8, 4, 2 or 1
  bool flat;         // aligned 16-byte granules with per-row-lane column shifts (B's rows are not
                     // 16-byte aligned); units then counts one granule more than the block's columns
  int units;         // column units (of `vec` columns) per thread block
  int row_lanes;     // k rows visited per pass of a thread block
  int threads;       // launch width (multiple of 32, >= units * row_lanes)
  int col_blocks;    // thread blocks along n
  int split_k;       // thread blocks along k
  int64_t k_per_split;
  int k_chunk;       // k rows of A staged in shared memory at a time
  size_t smem_bytes;
  size_t workspace_bytes;  // partial sums [split_k][b][m][n] f32 when split_k > 1
};

// Chooses the decomposition for rows [0, m) with m <= 16.  split_k 0 = automatic.
SkinnyPlan skinny_plan(int sms, int64_t b, int m, int64_t k, int64_t n, int vec, int split_k);

// Largest vector width (in bf16 elements) the operands' alignment and n allow.
int skinny_vec(int64_t n, const void* B);

// Enqueues C[:, i0:i0+m, :] += A[:, i0:i0+m, :] x B for m <= 16 (one row chunk).
// a_batch / c_batch are the batch strides in elements of the full tensors.
cudaError_t skinny_launch(const SkinnyPlan& plan, int64_t b, int m, int64_t k, int64_t n,
                          const uint16_t* A, int64_t a_batch, const uint16_t* B, float* C,
                          int64_t c_batch, float* workspace, cudaStream_t stream,
                          uint64_t* launches, bool overwrite = false);

// Enqueues the slice-ordered reduce: C[b, i, :] += partial[0] + partial[1] + ... for the
// b * m * n sums of one row chunk (partial is [split_k][b][m][n], c_batch the batch stride of C).
// c_cols > 0: C is dense [b][m][c_cols] with c_cols <= n; the columns of the partial sums past
// c_cols (sums over zero padding) are dropped.
cudaError_t skinny_reduce_launch(const float* partial, float* C, int64_t b, int m, int64_t n,
                                 int64_t c_batch, int split_k, cudaStream_t stream,
                                 bool overwrite = false, int64_t c_cols = 0);

// ---- streaming GEMV (FP32 FMA, B through a TMA ring, m <= 4) ------------------
struct StreamPlan {
  bool supported;
  int m_tile;        // 1, 2 or 4
  int strips;        // thread blocks along n (64 columns each)
  int split_k;       // thread blocks along k
  int k_per_split;   // multiple of the box height
  bool cluster_k;    // the slices of a strip are one cluster and add up through distributed
                     // shared memory: one launch, no scratch (2 <= split_k <= 8)
  size_t smem_bytes;
  size_t workspace_bytes;  // partial sums [split_k][b][m][n] f32 when the reduce kernel adds them
};
// Needs n % 8 == 0 and a 16-byte-aligned B (the TMA engine addresses B through a tensor map).
bool stream_shape_supported(int64_t b, int m, int64_t k, int64_t n, const void* B);
StreamPlan stream_plan(int sms, int64_t b, int m, int64_t k, int64_t n, int split_k,
                       bool scratch_reduce = false);
cudaError_t stream_launch(const DeviceInfo& dev, const StreamPlan& plan, int64_t b, int m, int64_t k,
                          int64_t n, const uint16_t* A, int64_t a_batch, const uint16_t* B, float* C,
                          int64_t c_batch, float* workspace, cudaStream_t stream,
                          uint64_t* launches, bool overwrite = false);

// ---- float32 inputs: split into bf16 terms laid side by side along k ----------
// Bytes of the buffer that holds A6[b][m][6k] and B6[b][6k][n] (bf16).
size_t f32_split_bytes(int64_t b, int64_t m, int64_t k, int64_t n);
// Enqueues the two split kernels; *A6 and *B6 point into `split` afterwards.
cudaError_t f32_split_launch(int64_t b, int64_t m, int64_t k, int64_t n, const float* A, const float* B,
                             void* split, bool six, uint16_t** A6, uint16_t** B6, cudaStream_t stream,
                             uint64_t* launches);

// ---- zero-padded copies of operands the TMA engine cannot address --------------
struct PadPlan {
  int64_t k8, n8;                    // k and n rounded up to multiples of 8
  bool stage_a, stage_b;             // which operands go through a padded copy
  bool stage_c;                      // C's rows are not TMA-addressable: the kernels write them
                                     // from registers (no copy of C is made)
  size_t bytes_a, bytes_b;           // sizes of the copies in the workspace (multiples of 256)
};
// Which operands need a copy for these extents and pointers.
PadPlan pad_plan(int64_t b, int64_t m, int64_t k, int64_t n, const void* A, const void* B,
                 const void* C);
cudaError_t pad_operands_launch(const PadPlan& p, int64_t b, int64_t m, int64_t k, int64_t n,
                                const uint16_t* A, const uint16_t* B, uint16_t* A_pad,
                                uint16_t* B_pad, cudaStream_t stream, uint64_t* launches);

// ---- tcgen05 path ------------------------------------------------------------
struct GemmPlan {
  bool supported;
  int form;      // 1: one CTA per 128-row tile, 2: a CTA pair per 256-row tile
  int tile_n;    // 64, 128 or 256 columns per tile
  size_t workspace_bytes;
  bool halves;   // tiles of a sparse last wave may be cut into column halves
  int split_k;   // operand-swapped kernel only: k slices per strip, added inside a cluster (1, 2, 4, 8)
  int ws_split;  // > 1: k slices whose sums go to partial[slice][b][m][n] in the workspace and are
                 // added, slice by slice and then to C, by the reduce kernel
  int raster_g = 0;  // rows of tiles per group of the tile order; 0: a column of tiles at a time
};

bool gemm_shape_supported(int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                          const void* B, const void* C);
// `knob`: 0 = by shape; otherwise form + 16 * (tile columns / 64) [+ 256 to keep the last wave's
// tiles whole] [+ 512 * k slices through the workspace] [+ 8192 * rows of tiles per group of the
// tile order, 63 = a column of tiles at a time], every part 0 = by shape; with form 3 the second
// part is the number of k slices added inside a cluster (0 = by shape, 1, 2, 4 or 8).
GemmPlan gemm_plan(int sms, int64_t b, int64_t m, int64_t k, int64_t n, int knob);
// The k range as a sequence of up to 8 equal segments, each reading one of the stored k ranges
// of A and of B (float32 inputs: six products of three stored terms each, see f32_split.cu):
// segment s covers k blocks [s * blocks, (s + 1) * blocks) of the call and reads stored blocks
// term * blocks + ..., term = 3 bits of a_terms / b_terms at position 3 s.
struct KSegments {
  int blocks;            // 64-element k blocks per segment
  uint32_t a_terms, b_terms;
  int64_t k_stored;      // k extent of the stored A and B (terms x blocks x 64)
};
// CTA pairs (cta_group::2) the current device can hold at once.
int gemm_pair_units(int sms);
// b_layout: 0 = B row-major [b][k][n], 1 = column-major [b][n][k], a multiple of 64 = packed in
// strips of that many columns, [b][ceil(n / strip)][k][strip].
// c_cols: 0 = C is [b][m][n] and 16-byte aligned (addressed by the TMA engine); otherwise C is
// [b][m][c_cols] with c_cols <= n (B carries n - c_cols columns of zero padding) and any 4-byte
// alignment, and is written from registers, element by element.
cudaError_t gemm_launch(const DeviceInfo& dev, const GemmPlan& plan, int64_t b, int64_t m,
                        int64_t k, int64_t n, const uint16_t* A, const uint16_t* B, float* C,
                        float* workspace, cudaStream_t stream, uint64_t* launches,
                        bool overwrite = false, int b_layout = 0, const KSegments* seg = nullptr,
                        int64_t c_cols = 0);

// ---- B stored column-major where the TMA engine cannot address it ------------
// C[b, i, j] (+)= sum_p A[b, i, p] * Bt[b, j, p]: one warp per output column, lanes stride over
// k, shuffle sums in a fixed order.  Any shape, no alignment needs; slow, deterministic.
cudaError_t colmajor_fallback_launch(int64_t b, int64_t m, int64_t k, int64_t n, const uint16_t* A,
                                     const uint16_t* Bt, float* C, bool overwrite,
                                     cudaStream_t stream, uint64_t* launches);

// ---- B packed in strips where the tensor kernels cannot run --------------------
// C[b, i, j] (+)= sum_p A[b, i, p] * Bp[b][j / strip][p][j mod strip]: one thread per output
// element.  Any strip and shape, no alignment needs; slow, deterministic.
cudaError_t packed_fallback_launch(int64_t strip, int64_t b, int64_t m, int64_t k, int64_t n,
                                   const uint16_t* A, const uint16_t* Bp, float* C, bool overwrite,
                                   cudaStream_t stream, uint64_t* launches);

// ---- bookkeeping shared with the other translation units' entry points (api.cu) ----------
// Adds to the count morello_launch_count() reports.
void count_launches(uint64_t launches);
// Records a failed CUDA call where morello_last_cuda_error() finds it, clears the runtime's
// sticky error and returns MORELLO_ERR_CUDA.
int record_cuda_error(cudaError_t e);

// ---- self-test of the bounded device-side waits --------------------------------
// One thread waits at most limit_ns on a barrier nothing arrives on, gives up, records the
// site in `status` and sets *gave_up (device memory) to 1.
cudaError_t wait_timeout_selftest_launch(uint32_t* status, uint64_t limit_ns, int* gave_up,
                                         cudaStream_t stream);

}  // namespace morello
