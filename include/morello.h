/*
 * morello.h -- C ABI of the B200 (sm_100a) MatmulAccum library.
 *
 * The operation is the paper's accumulating batched matrix multiply
 * (Section 2, "Tiling": dimensions are ordered batch, m, k, n and the output
 * is shaped batch x m x n; Section 2.2: MatmulAccum is the accumulating member
 * of the Matmul / MatmulAccum pair and its operands are typed bf16, bf16 and
 * f32; a bf16 -> f32 Move is an exact upcast):
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p<k} A[b,i,p] * B[b,p,j]
 *
 * Layout (unless an entry point says otherwise: B may also be given column-major or packed in
 * strips of columns, A and B as float32): dense row-major, no leading dimensions,
 *     A[b][m][k]  bf16   (read only)
 *     B[b][k][n]  bf16   (read only, one matrix per batch, no broadcasting)
 *     C[b][m][n]  f32    (read-modify-write)
 * Products are exact in f32; sums are accumulated in f32 (on the FP32 units or
 * in the tensor cores' f32 accumulators) in an order that is fixed for a given
 * shape and device, so repeated calls give identical bits.  C is added once,
 * after the sum over k is complete.
 *
 * Special values follow IEEE 754 as the definition's sum of products does: bf16
 * subnormal inputs and float32 subnormal sums are kept (no flush to zero), an
 * infinity or a NaN reaches exactly the elements of C whose sum contains it,
 * Inf x 0 and Inf - Inf give NaN.  Two exceptions.  (1) When C cannot be
 * addressed by the TMA engine (n % 8 != 0 or C not 16-byte aligned) and the
 * tile kernel (more than 64 rows) runs on padded copies, the final C + sum is a
 * reduction performed in L2, which treats a subnormal C, a subnormal sum and a
 * subnormal result as zero: an error of at most 2^-126 per element.  (2) The float32
 * entry point splits its inputs into bf16 terms; an infinite input turns every
 * result it reaches into NaN (the split forms Inf - Inf) where the definition
 * gives +-Inf.
 *
 * Ownership: the caller owns every buffer; the library keeps no reference to
 * them after the enqueued work has run.  C must not overlap A, B or the
 * workspace (not checked).  Unless stated otherwise pointers are DEVICE
 * pointers on the current CUDA device, calls are asynchronous on `stream`
 * (a cudaStream_t passed as void*; NULL is the legacy default stream) and
 * never synchronise the host.
 *
 * Errors: the int return value (a morello_status_t) is the only channel.  On
 * any error nothing is enqueued.  There is no CPU fallback: a device that is
 * not compute capability 10.x yields MORELLO_ERR_UNSUPPORTED_DEVICE.
 */
#ifndef MORELLO_H_
#define MORELLO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MORELLO_OK = 0,
  MORELLO_ERR_INVALID_SHAPE = 1,      /* a dimension < 0, or a byte size overflows int64 */
  MORELLO_ERR_NULL_POINTER = 2,       /* A, B or C null while its element count is > 0 */
  MORELLO_ERR_MISALIGNED = 3,         /* A or B not 2-byte aligned, C not 4-byte aligned,
                                         workspace not 16-byte aligned */
  MORELLO_ERR_UNSUPPORTED_DEVICE = 4, /* current device is not compute capability 10.x */
  MORELLO_ERR_WORKSPACE = 5,          /* workspace too small, or its allocation failed */
  MORELLO_ERR_CUDA = 6,               /* a CUDA call failed; see morello_last_cuda_error() */
  MORELLO_ERR_DEVICE_TIMEOUT = 7,     /* a bounded device-side wait gave up; only reported by
                                         morello_read_device_status() */
  MORELLO_ERR_UNSUPPORTED_PATH = 8    /* a forced path cannot run this shape / alignment */
} morello_status_t;

/* Kernel families behind the shape selector (Section 2 of the paper tiles one
 * MatmulAccum into smaller ones; here the tiling is fixed per family). */
enum {
  MORELLO_PATH_AUTO = -1,
  MORELLO_PATH_SKINNY = 0,  /* HBM-streaming FP32-FMA kernel, rows in chunks of <= 16 */
  MORELLO_PATH_TCGEN05 = 1  /* TMA + tcgen05 tensor-core GEMM with fused C += epilogue */
};

/*
 * MatmulAccum(b x m x k x n), the definition at the top of this file.
 * Any dimension may be 0: b*m*n == 0 or k == 0 returns MORELLO_OK with C
 * untouched (empty sum).  Scratch memory, when the chosen kernel needs any, is
 * a per-device buffer owned by the library that grows on demand (the only
 * allocation this call can make); concurrent calls on different streams that
 * both need scratch must use morello_matmul_accum_ws instead.  Growing the buffer
 * frees and allocates device memory, which a stream capture does not allow: a call
 * that would have to grow it while `stream` is being captured returns
 * MORELLO_ERR_WORKSPACE and touches nothing -- size the buffer with an ordinary call
 * on the same shape first, or capture morello_matmul_accum_ws.  The same holds for
 * every entry point below that uses the library's own buffers, and the library's first
 * call on a device (which allocates a 256-byte status block) must come before any capture.
 */
int morello_matmul_accum(int64_t b, int64_t m, int64_t k, int64_t n,
                         const void* A, const void* B, float* C, void* stream);

/*
 * Bytes of scratch that suffice for morello_matmul_accum_ws on this shape on the
 * current device, whatever the alignment of A, B and C turns out to be (the kernel
 * chosen depends on it): 0 if none can be needed; also 0 for invalid shapes.
 */
size_t morello_workspace_bytes(int64_t b, int64_t m, int64_t k, int64_t n);

/*
 * Same operation with caller-provided scratch: `workspace` is a device buffer
 * of `workspace_bytes` >= morello_workspace_bytes(...), 16-byte aligned (may be
 * NULL when 0 bytes are needed).  Its contents need no initialisation and are
 * unspecified afterwards.  Makes no allocation.
 */
int morello_matmul_accum_ws(int64_t b, int64_t m, int64_t k, int64_t n,
                            const void* A, const void* B, float* C,
                            void* workspace, size_t workspace_bytes, void* stream);

/*
 * Matmul(b x m x k x n), the non-accumulating member of the pair (Section 2.2 of the
 * paper lists Matmul beside MatmulAccum; Matmul is MatmulAccum into a zeroed output):
 *
 *     C[b,i,j]  <-  sum_{p<k} A[b,i,p] * B[b,p,j]
 *
 * Same layouts, kernels, scratch rules and status codes as morello_matmul_accum.  C is
 * write-only: its prior contents are neither read nor added (the kernels skip the read,
 * which on large outputs is a third of the memory traffic).  k == 0 sets C to zero;
 * b*m*n == 0 does nothing.
 */
int morello_matmul(int64_t b, int64_t m, int64_t k, int64_t n,
                   const void* A, const void* B, float* C, void* stream);

/* morello_matmul on a given path / split / tile: arguments as morello_matmul_accum_forced. */
int morello_matmul_forced(int path, int split_k,
                          int64_t b, int64_t m, int64_t k, int64_t n,
                          const void* A, const void* B, float* C,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * MatmulAccum with B stored column-major (layouts are a field of the paper's Spec; its
 * example in Section 2.2, a 1x4x128x16 Matmul, has a col_major right-hand side):
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p<k} A[b,i,p] * Bt[b,j,p],    Bt[b][n][k] bf16, k contiguous
 *
 * A and C as everywhere else.  With k % 8 == 0, n % 8 == 0 and 16-byte-aligned pointers the
 * tensor-core kernels run it (for them a column-major B is the K-major operand; `tile` is
 * their tile selector as in morello_matmul_accum_forced, 0 = by shape); any other shape
 * runs on a plain one-warp-per-column kernel.  Scratch as in morello_matmul_accum.  Same status
 * codes, asynchronous on `stream`, deterministic.
 */
int morello_matmul_accum_colmajor_b(int tile, int64_t b, int64_t m, int64_t k, int64_t n,
                                    const void* A, const void* Bt, float* C, void* stream);

/*
 * MatmulAccum with B in a packed layout (Section 2.4.2 of the paper: a layout may carry a strip
 * dimension of size s on a logical dimension -- Goto-style packing): the columns of B are cut
 * into strips of `strip`, each strip stored row-major and the strips one after another,
 *
 *     Bp[b][ceil(n / strip)][k][strip] bf16,    B[b,p,j] = Bp[b][j / strip][p][j mod strip]
 *
 * (the last strip is padded to `strip` columns; the padding is never used, whatever it holds).
 *
 *     C[b,i,j]  <-  C[b,i,j] + sum_{p<k} A[b,i,p] * B[b,p,j]
 *
 * A and C as everywhere else.  With strip % 64 == 0, k % 8 == 0, n % 8 == 0 and 16-byte-aligned
 * pointers the tensor-core kernels run it (a 64-column box of a strip is one contiguous 8 KiB
 * read); anything else runs on a plain one-thread-per-output kernel.  strip == 1 is the
 * column-major layout.  Scratch as in morello_matmul_accum.  Same status codes, asynchronous on
 * `stream`, deterministic.
 */
int morello_matmul_accum_packed_b(int strip, int64_t b, int64_t m, int64_t k, int64_t n,
                                  const void* A, const void* Bp, float* C, void* stream);

/* Matmul (C = A x B, C never read; k == 0 sets C to zero) with B column-major or packed:
 * arguments, kernels and status codes as the two accumulating entry points above. */
int morello_matmul_colmajor_b(int tile, int64_t b, int64_t m, int64_t k, int64_t n,
                              const void* A, const void* Bt, float* C, void* stream);
int morello_matmul_packed_b(int strip, int64_t b, int64_t m, int64_t k, int64_t n,
                            const void* A, const void* Bp, float* C, void* stream);

/*
 * MatmulAccum on float32 inputs (the paper's other benchmark, Section 7, is a float32
 * 2048-square matrix multiplication): A[b][m][k], B[b][k][n] and C[b][m][n] all f32, dense
 * row-major device pointers, 4-byte aligned; C += A x B.
 * Each float is split exactly into three bf16 terms and the six largest of the nine cross
 * products are computed by the bf16 kernels in one MatmulAccum(b, m, 6k, n) (the dropped
 * terms are below 2^-23 of |a*b|), so the result meets the same acceptance rule as the bf16
 * operation, is deterministic, and is exact when the inputs are bf16-representable.  The
 * split operands (12 bytes per element of A and B) live in a per-device buffer owned by
 * the library that grows on demand (the call may allocate, and synchronises the device when
 * it has to grow the buffer); concurrent calls on different streams share that buffer and
 * must be serialised by the caller.  Meant for GEMM-shaped problems: with few rows the
 * split of B costs more than the multiply.  Finite inputs only.
 */
int morello_matmul_accum_f32(int64_t b, int64_t m, int64_t k, int64_t n,
                             const float* A, const float* B, float* C, void* stream);

/* Matmul on float32 inputs: C = A x B, C never read (k == 0 sets C to zero); otherwise as
 * morello_matmul_accum_f32. */
int morello_matmul_f32(int64_t b, int64_t m, int64_t k, int64_t n,
                       const float* A, const float* B, float* C, void* stream);

/*
 * End-to-end convenience call on HOST buffers (same layouts): copies A, B and
 * C to library-owned device staging (one buffer per device, grown on demand), runs
 * the operation, copies C back and synchronises before returning.  Pinned host memory
 * makes the copies asynchronous with respect to each other but the call still
 * returns only when C_host holds the result.  Host threads that call it at the same
 * time take turns inside the library (the staging buffer is shared), so it is safe
 * but not concurrent.
 */
int morello_matmul_accum_host(int64_t b, int64_t m, int64_t k, int64_t n,
                              const void* A_host, const void* B_host, float* C_host);

/*
 * Allocation-free variant (the paper has no counterpart: this exists for callers,
 * not for the method).  Same operation, computed by the FP32-FMA kernel with the k
 * range cut into `split_k` slices (0 = let the library choose); the slices' partial
 * sums go to a fixed device array of MORELLO_NOALLOC_SCRATCH_BYTES that is part of
 * the library image, so neither this call nor anything it uses calls cudaMalloc,
 * cudaFree or an allocating library routine.  It is meant for processes that must not
 * allocate at call time: ones that gave all device memory to their own pool at
 * start-up (a late cudaMalloc may fail there, and while it runs it holds up every
 * stream of the process), or ones barred from growing their footprint once serving.
 *
 * Limits and rules:
 *  - the partial sums, split_k * b * min(m, 16) * n * 4 bytes, must fit the array;
 *    otherwise MORELLO_ERR_WORKSPACE is returned and nothing is enqueued
 *    (split_k = 1 needs no scratch and always fits);
 *  - the first call on each device resolves the array's device address (with that
 *    device current) and queries two device attributes; make that first call before
 *    starting any stream capture.  The CUDA runtime may load a kernel's code onto the
 *    device the first time that kernel is launched (lazy module loading), which is an
 *    allocation of the runtime's, not of this library: after one warm-up call per kernel
 *    variant (row count 1, 2, 4, 8 or 16 of the last chunk, load width, aligned or
 *    shifted-granule form) -- or with CUDA_MODULE_LOADING=EAGER -- no call changes the
 *    device's free memory;
 *  - all calls on a device share the one array and it keeps whatever the last call
 *    left in it.  Nothing in it has to be zero beforehand (every word that is read was
 *    written by the same call), but two calls that overlap on the GPU -- different
 *    streams, or one stream of each of two host threads -- race on it: serialise them;
 *  - every GPU that loads the library holds the array until the process exits.
 * Otherwise as morello_matmul_accum: device pointers, asynchronous on `stream`, same
 * status codes, deterministic for a given shape and split.
 */
#define MORELLO_NOALLOC_SCRATCH_BYTES (4u << 20)
int morello_matmul_accum_noalloc(int split_k, int64_t b, int64_t m, int64_t k, int64_t n,
                                 const void* A, const void* B, float* C, void* stream);

/* MORELLO_NOALLOC_SCRATCH_BYTES as the loaded library was built with. */
size_t morello_noalloc_scratch_limit(void);

/* --- introspection and experiments (tests and benchmarks) ------------------ */

/* The path the selector picks for this shape with 16-byte-aligned operands:
 * MORELLO_PATH_SKINNY or MORELLO_PATH_TCGEN05 (-1 for an invalid shape).  A single row
 * (the GEMV) goes to the FP32-FMA kernels when its 64-column strips fill the device's block
 * slots about once and k is short (the 1 x 2048 x 16384 case), or when B is small or not
 * addressable by the TMA engine, and to the operand-swapped tcgen05 kernel otherwise (it
 * streams long or many-strip B faster); from 2 rows on the tcgen05 kernels run whenever they can
 * address the shape (k % 8 == 0, n % 8 == 0); other extents with at least 2 rows reach them
 * through zero-padded copies of the operands in the workspace whenever that is estimated to
 * cost less than the FMA kernels, which stream B once per 16 rows (also reported as
 * MORELLO_PATH_TCGEN05; forcing that path means the direct kernels and refuses such
 * shapes).  (The single-row choice looks at the device's SM count;
 * 148 SMs are assumed when no device is usable). */
int morello_select_path(int64_t b, int64_t m, int64_t k, int64_t n);

/*
 * Which kernel, tile and k slices morello_matmul_accum would use for this shape with 16-byte-
 * aligned operands on the current device (148 SMs assumed when no device is usable), as one line
 * of text for logs: e.g. "tcgen05 gemm_kernel: a CTA pair per 256 x 256 tile, ...".  `text`
 * (host memory, `text_bytes` long, caller-owned) receives at most text_bytes - 1 characters and
 * a terminating NUL.  Enqueues nothing.  Returns MORELLO_OK, MORELLO_ERR_NULL_POINTER for a
 * missing buffer, or MORELLO_ERR_INVALID_SHAPE.  With MORELLO_LOG=1 in the environment when the
 * library is first used, every call that goes through the selector prints this line on stderr.
 */
int morello_describe_route(int64_t b, int64_t m, int64_t k, int64_t n, char* text, size_t text_bytes);

/*
 * Run on a given path (MORELLO_PATH_AUTO = selector) with a given split of the
 * k range across thread blocks (0 = automatic).  On the skinny path (value % 1024) is
 * that split and (value / 1024) picks the kernel: 0 = by shape, 1 = the register-
 * streaming kernel (any shape), 2 = the TMA-ring GEMV kernel (m <= 4, n % 8 == 0,
 * 16-byte-aligned B; it raises the split as needed to keep the part of A a block
 * stages within 32 KiB: 16384 / m rows of k per block, m rounded up to 1, 2 or 4; up to
 * 8 slices are added inside a thread-block cluster, without scratch), 3 = the same kernel
 * with the slices always added by the reduce kernel from scratch.  On the tcgen05 path the
 * argument instead selects the tile: (value % 16) is the form -- 0 = by
 * shape, 1 = one CTA per 128-row tile, 2 = a pair of CTAs per 256-row tile
 * (cta_group::2), 3 = the operand-swapped kernel for at most 64 rows (with it the next
 * field is the number of k slices added inside a cluster instead: 0 = by shape, 1, 2, 4, 8) -- ((value / 16) % 16) is the tile's column count / 64 -- 0 = by
 * shape, 1, 2 or 4 (64 columns only with form 1) -- adding 256 keeps the tiles of a
 * sparse last wave whole instead of cutting them into column halves, and ((value / 512) % 16)
 * is the number of k slices whose partial sums go through the workspace (slices x b x m x n x 4
 * bytes) and are added in slice order, then to C, by one more launch: 0 = by shape (only
 * calls whose tiles fill less than half the device and whose k spans at least 32 blocks of 64
 * are cut), 1 = none, 2 .. 8 (fewer are used if a slice would be empty or the sums would
 * exceed 64 MiB), and ((value / 8192) % 64) is the tile order: tiles are walked in groups of that
 * many rows of tiles, row-fastest inside a group, so that the tiles in flight share a few rows of
 * A and a few columns of B (0 = by shape, which is 8; 63 = a whole column of tiles at a time).
 * Returns MORELLO_ERR_UNSUPPORTED_PATH, and
 * enqueues nothing, when the path cannot run the shape (the tcgen05 path needs
 * k % 8 == 0, n % 8 == 0 and 16-byte-aligned A, B, C) or the value names no tile.
 * workspace may be NULL with workspace_bytes 0 to use the library's own per-device
 * scratch.
 */
int morello_matmul_accum_forced(int path, int split_k,
                                int64_t b, int64_t m, int64_t k, int64_t n,
                                const void* A, const void* B, float* C,
                                void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch the forced variant needs for this path and split. */
size_t morello_workspace_bytes_forced(int path, int split_k,
                                      int64_t b, int64_t m, int64_t k, int64_t n);

/*
 * Synchronises `stream`, then reads and clears the device-side status word
 * that bounded waits inside the kernels write when they give up.  Returns
 * MORELLO_OK, MORELLO_ERR_DEVICE_TIMEOUT or MORELLO_ERR_CUDA.  If `detail` is
 * not NULL it receives the raw status word (0 when OK).
 */
int morello_read_device_status(void* stream, uint32_t* detail);

/*
 * Self-test of the bounded device-side waits (every mbarrier wait in the kernels gives up
 * after a time limit -- 2 s in the kernels proper -- records where in the status word and lets
 * its block return, so a stalled pipeline becomes an error code, not a hung device).  Launches
 * one thread that waits at most `limit_ms` (1 .. 1000) on a barrier that nothing arrives on,
 * and synchronises `stream`.  Returns MORELLO_OK when the wait gave up as designed (the status
 * word is then set: the next morello_read_device_status returns MORELLO_ERR_DEVICE_TIMEOUT and
 * clears it), MORELLO_ERR_CUDA if it did not.  Faults and hangs nothing.
 */
int morello_selftest_wait_timeout(uint32_t limit_ms, void* stream);

/*
 * Host-only self-test of the once-per-device bookkeeping (function attributes such as the
 * shared-memory opt-in belong to each device's copy of a kernel, so they are set once per
 * device, not once per process): simulates `calls_per_device` rounds of calls over `devices`
 * device indices, the first set-up attempt on device 1 failing, and returns how often the
 * set-up ran -- `devices` + 1 when devices >= 2 and calls_per_device >= 2 (a failure is
 * retried, a success is remembered).  Needs no GPU; -1 for negative arguments.
 */
int morello_selftest_per_device_once(int devices, int calls_per_device);

/*
 * What the kernels size their grids by on the current device: the number of SMs and
 * the number of two-CTA clusters (cta_group::2 pairs) the device can hold at once,
 * which may be fewer than half the SMs.  Either pointer may be NULL.
 */
int morello_device_limits(int* sms, int* cta_pairs);

/* Kernel launches enqueued by this library since it was loaded (all devices). */
uint64_t morello_launch_count(void);

/* The cudaError_t of the most recent failed CUDA call on this thread (0 if none). */
int morello_last_cuda_error(void);

/* Static, NUL-terminated description of a status code. */
const char* morello_status_string(int status);

/* Static version string. */
const char* morello_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MORELLO_H_ */
