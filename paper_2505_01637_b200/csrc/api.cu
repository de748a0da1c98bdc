// C ABI of the library: argument validation, per-device state, the shape
// selector and the dispatch to the two kernel families.
#include <algorithm>
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "../../include/morello.h"
#include "internal.h"

namespace morello {
namespace {

constexpr int kMaxDevices = 64;
constexpr int kSkinnyMaxRows = 16;

struct DeviceState {
  bool ready = false;
  int status_code = MORELLO_OK;  // result of the one-time set-up
  DeviceInfo info;
  void* scratch = nullptr;       // library-owned workspace, grown on demand
  size_t scratch_bytes = 0;
  void* stage = nullptr;         // device staging for the host-buffer entry point
  size_t stage_bytes = 0;
  void* split = nullptr;         // bf16 terms of float32 operands (morello_matmul_accum_f32)
  size_t split_bytes = 0;
};

std::mutex g_mutex;
DeviceState g_dev[kMaxDevices];
std::atomic<uint64_t> g_launches{0};
thread_local int t_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
  t_last_cuda_error = (int)e;
  (void)cudaGetLastError();
  return MORELLO_ERR_CUDA;
}

// The library-owned buffers grow by freeing and allocating, which is illegal while `stream` is
// being captured into a graph (it would invalidate the capture): such a call is refused
// instead, before anything touches the device.
bool capturing(cudaStream_t stream) {
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) {
    (void)cudaGetLastError();
    return false;
  }
  return st != cudaStreamCaptureStatusNone;
}

// One-time set-up per device, under g_mutex.
int device_state(DeviceState** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return MORELLO_ERR_UNSUPPORTED_DEVICE;
  DeviceState& st = g_dev[dev];
  if (!st.ready) {
    int major = 0, sms = 0;
    if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess)
      return cuda_fail(e);
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
      return cuda_fail(e);
    st.info.cc_major = major;
    st.info.sms = sms;
    if (major != 10) {
      st.status_code = MORELLO_ERR_UNSUPPORTED_DEVICE;
    } else {
      if ((e = cudaMalloc((void**)&st.info.status, 256)) != cudaSuccess) return cuda_fail(e);
      if ((e = cudaMemset(st.info.status, 0, 256)) != cudaSuccess) return cuda_fail(e);
      st.status_code = MORELLO_OK;
    }
    st.ready = true;
  }
  *out = &st;
  return st.status_code;
}

// Bounded text output for morello_describe_route.
struct TextOut {
  char* text;
  size_t bytes, at;
  __attribute__((format(printf, 2, 3))) void append(const char* fmt, ...) {
    if (at + 1 >= bytes) return;
    va_list ap;
    va_start(ap, fmt);
    const int w = vsnprintf(text + at, bytes - at, fmt, ap);
    va_end(ap);
    if (w > 0) at = std::min(bytes - 1, at + (size_t)w);
  }
};

bool mul_overflows(int64_t a, int64_t b, int64_t* out) {
  return __builtin_mul_overflow(a, b, out);
}

// Shape and pointer checks common to every entry point.  Sets *empty when there
// is nothing to do.
int validate(int64_t b, int64_t m, int64_t k, int64_t n, const void* A, const void* B,
             const void* C, bool* empty) {
  *empty = false;
  if (b < 0 || m < 0 || k < 0 || n < 0) return MORELLO_ERR_INVALID_SHAPE;
  int64_t mk, kn, mn, t;
  if (mul_overflows(m, k, &mk) || mul_overflows(k, n, &kn) || mul_overflows(m, n, &mn) ||
      mul_overflows(b, mk, &t) || mul_overflows(t, 2, &t) || mul_overflows(b, kn, &t) ||
      mul_overflows(t, 2, &t) || mul_overflows(b, mn, &t) || mul_overflows(t, 4 * 64, &t))
    return MORELLO_ERR_INVALID_SHAPE;
  if (b == 0 || m == 0 || n == 0 || k == 0) {
    *empty = true;
    return MORELLO_OK;
  }
  if (!A || !B || !C) return MORELLO_ERR_NULL_POINTER;
  if (reinterpret_cast<uintptr_t>(A) % 2 || reinterpret_cast<uintptr_t>(B) % 2 ||
      reinterpret_cast<uintptr_t>(C) % 4)
    return MORELLO_ERR_MISALIGNED;
  return MORELLO_OK;
}

// Every extra row costs the FMA kernels one FMA per element of B while the tensor cores take
// the rows for free, so the FMA kernels keep the single row (the GEMV proper) and whatever the
// TMA engine cannot address; from two rows on the tensor path wins, few columns included (it
// cuts a long k into slices of its own when the columns alone cannot occupy the device).
constexpr int kFmaMaxRows = 1;
int select_path(int sms, int64_t b, int64_t m, int64_t k, int64_t n, const void* A, const void* B,
                const void* C) {
  if (!gemm_shape_supported(b, m, k, n, A, B, C)) return MORELLO_PATH_SKINNY;
  if (m <= kFmaMaxRows) {
    // The single row.  The FMA GEMV kernel is at its best when its 64-column strips (times its
    // k slices) fill the two block slots per SM exactly once and k is short; elsewhere the
    // operand-swapped tensor kernel streams B faster (128-column strips, deeper ring).  Below
    // 16 MB of B both finish within a launch latency or two and the FMA kernels are the lighter
    // launch.
    if (b > 65535 || b * k * n < (1ll << 23) || !stream_shape_supported(b, 1, k, n, B))
      return MORELLO_PATH_SKINNY;
    const StreamPlan pl = stream_plan(sms, b, 1, k, n, 0);
    if (!pl.supported) return MORELLO_PATH_TCGEN05;
    const int64_t blocks = b * pl.strips * pl.split_k, slots = 2ll * sms;
    const bool one_full_wave = blocks <= slots && blocks * 5 >= slots * 4;
    if (one_full_wave && (k <= 2048 || (b * pl.strips <= 128 && k <= 16384))) return MORELLO_PATH_SKINNY;
    return MORELLO_PATH_TCGEN05;
  }
  return MORELLO_PATH_TCGEN05;
}

// Extents the TMA engine cannot address (k % 8 != 0 or n % 8 != 0): the FMA kernels take the
// rows in chunks of 16 and stream B once per chunk; the padded-copy route pays one pass over the
// operands that need a copy and a launch or two more, and then runs at tensor-core speed.
// Estimated cost of both, in microseconds (the constants are fits to measurements on a B200);
// pointers that are merely misaligned keep the FMA route (the workspace a shape may need must
// not depend on them).
bool staged_wins(int64_t b, int64_t m, int64_t k, int64_t n) {
  if ((k % 8 == 0 && n % 8 == 0) || m < 2) return false;
  const int64_t limit = (1ll << 31) - 8;   // tensor-map extents are 32-bit
  if (b >= limit || m >= limit || k >= limit || n >= limit) return false;
  const double bytes_a = 2.0 * b * m * k, bytes_b = 2.0 * b * k * n, bytes_c = 4.0 * b * m * n;
  // The FMA kernel's cost per MB of B for a chunk of r rows: bound by memory up to a few rows,
  // then by one FMA per row and element.  Its flat form reads unaligned rows in aligned
  // 16-byte granules; tiny shapes fall back to narrow loads, which cost more of both.
  const bool flat = k >= 64 && n >= 16;
  const int vec = n % 8 == 0 ? 8 : n % 4 == 0 ? 4 : n % 2 == 0 ? 2 : 1;
  const double base = flat ? 0.25 : vec == 8 ? 0.2 : vec == 4 ? 0.3 : vec == 2 ? 0.37 : 0.5;
  const double per_row = flat ? 0.074 : vec == 8 ? 0.083 : vec == 4 ? 0.09 : vec == 2 ? 0.13 : 0.3;
  const double mb_b = bytes_b / 1e6;
  const int64_t full_chunks = m / 16, rest = m % 16;
  double fma = (double)full_chunks * (5.0 + mb_b * std::max(base, 16 * per_row));
  if (rest) fma += 5.0 + mb_b * std::max(base, (double)rest * per_row);
  // Copies in and out, then the tensor-core call itself: its FLOPs or its pass over memory.
  const double staged = 9.0 + (2.0 * (bytes_a + bytes_b) + 0.5 * bytes_c) / 4.4e6 +
                        std::max(2.0 * b * m * k * n / 1e9, (bytes_a + bytes_b + 2.0 * bytes_c) / 6e6);
  return staged < fma;
}

// Bytes of the padded-copy route's workspace when every operand is staged, its own tensor-core
// call included.
size_t staged_workspace(int sms, int64_t b, int64_t m, int64_t k, int64_t n) {
  const void* odd = reinterpret_cast<const void*>(uintptr_t(4100));   // 4-byte aligned only
  const PadPlan pp = pad_plan(b, m, k, n, odd, odd, odd);
  return pp.bytes_a + pp.bytes_b + gemm_plan(sms, b, m, pp.k8, pp.n8, 0).workspace_bytes;
}

// The knob of the forced entry point on the skinny path: knob % 1024 is the split of the k
// range (0 = automatic), knob / 1024 picks the kernel (0 = by shape, 1 = the register-
// streaming kernel, 2 = the TMA-ring GEMV kernel, which needs m <= 4, n % 8 == 0 and a
// 16-byte-aligned B, 3 = the same with the k slices always added by the reduce kernel from
// scratch instead of inside a cluster).
constexpr int kKnobSplitMod = 1024;
enum { SKINNY_AUTO = 0, SKINNY_REGISTER = 1, SKINNY_STREAM = 2, SKINNY_STREAM_SCRATCH = 3 };
inline bool knob_scratch_reduce(int knob) { return knob / kKnobSplitMod == SKINNY_STREAM_SCRATCH; }

// Which skinny kernel runs this shape: -1 = the request cannot be met.
int skinny_kernel_for(int knob, int64_t b, int64_t m, int64_t k, int64_t n, const void* B) {
  const int want = knob / kKnobSplitMod;
  const bool can = m <= 4 && stream_shape_supported(b, (int)m, k, n, B) &&
                   stream_plan(1, b, (int)m, k, n, knob % kKnobSplitMod).supported;
  if (want == SKINNY_REGISTER) return SKINNY_REGISTER;
  if (want == SKINNY_STREAM || want == SKINNY_STREAM_SCRATCH) return can ? SKINNY_STREAM : -1;
  if (want != SKINNY_AUTO) return -1;
  // Small problems finish inside one launch latency either way; the ring pays off once
  // there is a stream of B worth pipelining.
  return (can && k >= 256 && n >= 256) ? SKINNY_STREAM : SKINNY_REGISTER;
}

// Scratch for the skinny path over all row chunks (chunks run one after another on
// the stream, so they share the buffer).
size_t skinny_workspace(int sms, int64_t b, int64_t m, int64_t k, int64_t n, const void* B, int knob) {
  const int split_k = knob % kKnobSplitMod;
  const int which = skinny_kernel_for(knob, b, m, k, n, B);
  if (which == SKINNY_STREAM)
    return stream_plan(sms, b, (int)m, k, n, split_k, knob_scratch_reduce(knob)).workspace_bytes;
  const int vec = skinny_vec(n, B);
  // Chunks are full (16 rows) except possibly the last one.
  const int first = (int)std::min<int64_t>(kSkinnyMaxRows, m);
  size_t need = skinny_plan(sms, b, first, k, n, vec, split_k).workspace_bytes;
  const int last = (int)(m % kSkinnyMaxRows);
  if (m > kSkinnyMaxRows && last != 0)
    need = std::max(need, skinny_plan(sms, b, last, k, n, vec, split_k).workspace_bytes);
  return need;
}

size_t workspace_for(int sms, int path, int knob, int64_t b, int64_t m, int64_t k, int64_t n,
                     const void* B) {
  if (path == MORELLO_PATH_TCGEN05) return gemm_plan(sms, b, m, k, n, knob).workspace_bytes;
  return skinny_workspace(sms, b, m, k, n, B, knob);
}

// MORELLO_LOG=1 in the environment: every call through the selector prints the route it takes
// (the line morello_describe_route gives for the shape) on stderr.
void log_route(int path, int64_t b, int64_t m, int64_t k, int64_t n, bool overwrite, int b_layout) {
  static const bool on = [] {
    const char* v = getenv("MORELLO_LOG");
    return v && v[0] && v[0] != '0';
  }();
  if (!on) return;
  char text[256];
  if (path != MORELLO_PATH_AUTO || b_layout != 0)
    snprintf(text, sizeof text, "%s", b_layout ? "B column-major or packed: tensor kernels when addressable, else the plain fallback"
                                               : "forced path");
  else if (morello_describe_route(b, m, k, n, text, sizeof text) != MORELLO_OK)
    snprintf(text, sizeof text, "(no route)");
  fprintf(stderr, "morello: %s b=%lld m=%lld k=%lld n=%lld -> %s\n", overwrite ? "matmul" : "matmul_accum",
          (long long)b, (long long)m, (long long)k, (long long)n, text);
}

int run(int path, int split_k, int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
        const void* B, float* C, void* workspace, size_t workspace_bytes, bool own_scratch,
        void* stream, bool overwrite = false, int b_layout = 0,
        const KSegments* seg = nullptr) {
  bool empty = false;
  int rc = validate(b, m, k, n, A, B, C, &empty);
  if (rc != MORELLO_OK) return rc;
  log_route(path, b, m, k, n, overwrite, b_layout);
  if (split_k < 0) return MORELLO_ERR_INVALID_SHAPE;
  if (workspace && reinterpret_cast<uintptr_t>(workspace) % 16) return MORELLO_ERR_MISALIGNED;

  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK) return rc;
  if (empty) {
    // An empty sum: MatmulAccum leaves C alone, Matmul sets it to zero.
    if (overwrite && b > 0 && m > 0 && n > 0) {
      if (!C) return MORELLO_ERR_NULL_POINTER;
      if (reinterpret_cast<uintptr_t>(C) % 4) return MORELLO_ERR_MISALIGNED;
      const cudaError_t e = cudaMemsetAsync(C, 0, (size_t)b * m * n * 4, static_cast<cudaStream_t>(stream));
      if (e != cudaSuccess) return cuda_fail(e);
    }
    return MORELLO_OK;
  }

  // b_layout: 0 row-major B, 1 column-major, otherwise the strip size of a packed B.
  const bool b_col_major = b_layout != 0;     // any layout but row-major: tensor kernels or a fallback
  bool bt_fallback = false;
  bool staged = false;   // through zero-padded copies of the operands (see pad.cu)
  if (b_col_major) {
    // B as [b][n][k] or packed in strips: the tensor-core kernels when the TMA engine can
    // address the operands (a packed B needs strips that are multiples of their 64-column
    // boxes), else a plain kernel.  The FMA streaming kernels read B by rows only.
    if (path == MORELLO_PATH_SKINNY) return MORELLO_ERR_UNSUPPORTED_PATH;
    const bool tc = gemm_shape_supported(b, m, k, n, A, B, C) && (b_layout == 1 || b_layout % 64 == 0) &&
                    (b_layout == 1 || b * ((n + b_layout - 1) / b_layout) < (1ll << 31));
    if (path == MORELLO_PATH_TCGEN05 && !tc) return MORELLO_ERR_UNSUPPORTED_PATH;
    path = MORELLO_PATH_TCGEN05;
    bt_fallback = !tc;
  } else if (path == MORELLO_PATH_AUTO) {
    staged = staged_wins(b, m, k, n);
    path = staged ? MORELLO_PATH_TCGEN05 : select_path(st->info.sms, b, m, k, n, A, B, C);
  } else if (path == MORELLO_PATH_TCGEN05) {
    if (!gemm_shape_supported(b, m, k, n, A, B, C)) return MORELLO_ERR_UNSUPPORTED_PATH;
  } else if (path != MORELLO_PATH_SKINNY) {
    return MORELLO_ERR_UNSUPPORTED_PATH;
  }

  const int sms = st->info.sms;
  const int vec = skinny_vec(n, B);
  int which = SKINNY_REGISTER;
  if (path == MORELLO_PATH_SKINNY) {
    which = skinny_kernel_for(split_k, b, m, k, n, B);
    if (which < 0) return MORELLO_ERR_UNSUPPORTED_PATH;
  }
  PadPlan pad{};
  GemmPlan pad_gemm{};
  if (staged) {
    pad = pad_plan(b, m, k, n, A, B, C);
    pad_gemm = gemm_plan(sms, b, m, pad.k8, pad.n8, 0);
    if (!pad_gemm.supported) return MORELLO_ERR_UNSUPPORTED_PATH;
  }
  const size_t need = staged ? pad.bytes_a + pad.bytes_b + pad_gemm.workspace_bytes
                      : bt_fallback ? 0 : workspace_for(sms, path, split_k, b, m, k, n, B);
  float* ws = static_cast<float*>(workspace);
  if (need > 0) {
    if (own_scratch) {
      std::lock_guard<std::mutex> lock(g_mutex);
      if (st->scratch_bytes < need) {
        if (capturing(static_cast<cudaStream_t>(stream))) return MORELLO_ERR_WORKSPACE;
        // Work already enqueued may still be using the old buffer.
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) return cuda_fail(e);
        if (st->scratch) cudaFree(st->scratch);
        st->scratch = nullptr;
        st->scratch_bytes = 0;
        const size_t grow = std::max(need, (size_t)(8u << 20));
        if ((e = cudaMalloc(&st->scratch, grow)) != cudaSuccess) {
          cuda_fail(e);
          return MORELLO_ERR_WORKSPACE;
        }
        st->scratch_bytes = grow;
      }
      ws = static_cast<float*>(st->scratch);
    } else if (!ws || workspace_bytes < need) {
      return MORELLO_ERR_WORKSPACE;
    }
  }

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint64_t launches = 0;
  cudaError_t e = cudaSuccess;
  if (staged) {
    char* base = reinterpret_cast<char*>(ws);
    uint16_t* a_pad = reinterpret_cast<uint16_t*>(base);
    uint16_t* b_pad = reinterpret_cast<uint16_t*>(base + pad.bytes_a);
    float* inner_ws = reinterpret_cast<float*>(base + pad.bytes_a + pad.bytes_b);
    e = pad_operands_launch(pad, b, m, k, n, static_cast<const uint16_t*>(A),
                            static_cast<const uint16_t*>(B), a_pad, b_pad, s, &launches);
    if (e == cudaSuccess)
      e = gemm_launch(st->info, pad_gemm, b, m, pad.k8, pad.n8,
                      pad.stage_a ? a_pad : static_cast<const uint16_t*>(A),
                      pad.stage_b ? b_pad : static_cast<const uint16_t*>(B), C,
                      pad_gemm.workspace_bytes ? inner_ws : nullptr, s, &launches, overwrite, 0, nullptr,
                      pad.stage_c ? n : 0);
  } else if (bt_fallback && b_layout != 1) {
    e = packed_fallback_launch(b_layout, b, m, k, n, static_cast<const uint16_t*>(A),
                               static_cast<const uint16_t*>(B), C, overwrite, s, &launches);
  } else if (bt_fallback) {
    e = colmajor_fallback_launch(b, m, k, n, static_cast<const uint16_t*>(A),
                                 static_cast<const uint16_t*>(B), C, overwrite, s, &launches);
  } else if (path == MORELLO_PATH_TCGEN05) {
    const GemmPlan plan = gemm_plan(sms, b, m, k, n, split_k);
    if (!plan.supported) return MORELLO_ERR_UNSUPPORTED_PATH;
    e = gemm_launch(st->info, plan, b, m, k, n, static_cast<const uint16_t*>(A),
                    static_cast<const uint16_t*>(B), C, ws, s, &launches, overwrite, b_layout, seg);
  } else if (which == SKINNY_STREAM) {
    const StreamPlan plan = stream_plan(sms, b, (int)m, k, n, split_k % kKnobSplitMod,
                                        knob_scratch_reduce(split_k));
    e = stream_launch(st->info, plan, b, (int)m, k, n, static_cast<const uint16_t*>(A), m * k,
                      static_cast<const uint16_t*>(B), C, m * n, ws, s, &launches, overwrite);
  } else {
    const uint16_t* a = static_cast<const uint16_t*>(A);
    const int split = split_k % kKnobSplitMod;
    for (int64_t i0 = 0; i0 < m && e == cudaSuccess; i0 += kSkinnyMaxRows) {
      const int mc = (int)std::min<int64_t>(kSkinnyMaxRows, m - i0);
      const SkinnyPlan plan = skinny_plan(sms, b, mc, k, n, vec, split);
      e = skinny_launch(plan, b, mc, k, n, a + i0 * k, m * k, static_cast<const uint16_t*>(B),
                        C + i0 * n, m * n, ws, s, &launches, overwrite);
    }
  }
  g_launches.fetch_add(launches, std::memory_order_relaxed);
  if (e != cudaSuccess) return cuda_fail(e);
  return MORELLO_OK;
}

}  // namespace

void count_launches(uint64_t launches) { g_launches.fetch_add(launches, std::memory_order_relaxed); }
int record_cuda_error(cudaError_t e) { return cuda_fail(e); }

}  // namespace morello

using namespace morello;

#pragma GCC visibility push(default)
extern "C" {

int morello_matmul_accum(int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                         const void* B, float* C, void* stream) {
  return run(MORELLO_PATH_AUTO, 0, b, m, k, n, A, B, C, nullptr, 0, true, stream);
}

size_t morello_workspace_bytes(int64_t b, int64_t m, int64_t k, int64_t n) {
  // The selector looks at the pointers' alignment too, which is not known here: operands that
  // are not 16-byte aligned turn a tensor-core call into an FMA call, whose k slices need
  // scratch.  The answer covers every path the call could take.
  const size_t chosen = morello_workspace_bytes_forced(MORELLO_PATH_AUTO, 0, b, m, k, n);
  const size_t fma_register = morello_workspace_bytes_forced(MORELLO_PATH_SKINNY, kKnobSplitMod * SKINNY_REGISTER, b, m, k, n);
  const size_t fma_any = morello_workspace_bytes_forced(MORELLO_PATH_SKINNY, 0, b, m, k, n);
  return std::max(chosen, std::max(fma_register, fma_any));
}

size_t morello_workspace_bytes_forced(int path, int split_k, int64_t b, int64_t m, int64_t k,
                                      int64_t n) {
  bool empty = false;
  // A 16-byte-aligned stand-in address: only its alignment is looked at.
  const void* fake = reinterpret_cast<const void*>(uintptr_t(4096));
  if (validate(b, m, k, n, fake, fake, fake, &empty) != MORELLO_OK || empty || split_k < 0) return 0;
  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (device_state(&st) != MORELLO_OK) return 0;
  }
  if (path == MORELLO_PATH_AUTO && staged_wins(b, m, k, n))
    return staged_workspace(st->info.sms, b, m, k, n);
  if (path == MORELLO_PATH_AUTO) path = select_path(st->info.sms, b, m, k, n, fake, fake, fake);
  if (path == MORELLO_PATH_TCGEN05 && !gemm_shape_supported(b, m, k, n, fake, fake, fake)) return 0;
  if (path == MORELLO_PATH_SKINNY && skinny_kernel_for(split_k, b, m, k, n, fake) < 0) return 0;
  return workspace_for(st->info.sms, path, split_k, b, m, k, n, fake);
}

int morello_matmul_accum_ws(int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                            const void* B, float* C, void* workspace, size_t workspace_bytes,
                            void* stream) {
  return run(MORELLO_PATH_AUTO, 0, b, m, k, n, A, B, C, workspace, workspace_bytes, false, stream);
}

int morello_matmul_accum_forced(int path, int split_k, int64_t b, int64_t m, int64_t k, int64_t n,
                                const void* A, const void* B, float* C, void* workspace,
                                size_t workspace_bytes, void* stream) {
  const bool own = (workspace == nullptr && workspace_bytes == 0);
  return run(path, split_k, b, m, k, n, A, B, C, workspace, workspace_bytes, own, stream);
}

int morello_matmul(int64_t b, int64_t m, int64_t k, int64_t n, const void* A, const void* B,
                   float* C, void* stream) {
  return run(MORELLO_PATH_AUTO, 0, b, m, k, n, A, B, C, nullptr, 0, true, stream, true);
}

int morello_matmul_forced(int path, int split_k, int64_t b, int64_t m, int64_t k, int64_t n,
                          const void* A, const void* B, float* C, void* workspace,
                          size_t workspace_bytes, void* stream) {
  const bool own = (workspace == nullptr && workspace_bytes == 0);
  return run(path, split_k, b, m, k, n, A, B, C, workspace, workspace_bytes, own, stream, true);
}

int morello_matmul_accum_colmajor_b(int tile, int64_t b, int64_t m, int64_t k, int64_t n,
                                    const void* A, const void* Bt, float* C, void* stream) {
  if (tile < 0) return MORELLO_ERR_INVALID_SHAPE;
  return run(MORELLO_PATH_AUTO, tile, b, m, k, n, A, Bt, C, nullptr, 0, true, stream, false, true);
}

int morello_matmul_accum_packed_b(int strip, int64_t b, int64_t m, int64_t k, int64_t n,
                                  const void* A, const void* Bp, float* C, void* stream) {
  if (strip < 1) return MORELLO_ERR_INVALID_SHAPE;
  int64_t t;
  if (n > 0 && (mul_overflows((n + strip - 1) / strip, strip, &t) || mul_overflows(t, k > 0 ? k : 1, &t) ||
                mul_overflows(t, b > 0 ? b : 1, &t) || mul_overflows(t, 2, &t)))
    return MORELLO_ERR_INVALID_SHAPE;
  // A strip of one column is the column-major layout; the code 1 means exactly that below.
  return run(MORELLO_PATH_AUTO, 0, b, m, k, n, A, Bp, C, nullptr, 0, true, stream, false, strip);
}

int morello_matmul_colmajor_b(int tile, int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                              const void* Bt, float* C, void* stream) {
  if (tile < 0) return MORELLO_ERR_INVALID_SHAPE;
  return run(MORELLO_PATH_AUTO, tile, b, m, k, n, A, Bt, C, nullptr, 0, true, stream, true, 1);
}

int morello_matmul_packed_b(int strip, int64_t b, int64_t m, int64_t k, int64_t n, const void* A,
                            const void* Bp, float* C, void* stream) {
  if (strip < 1) return MORELLO_ERR_INVALID_SHAPE;
  int64_t t;
  if (n > 0 && (mul_overflows((n + strip - 1) / strip, strip, &t) || mul_overflows(t, k > 0 ? k : 1, &t) ||
                mul_overflows(t, b > 0 ? b : 1, &t) || mul_overflows(t, 2, &t)))
    return MORELLO_ERR_INVALID_SHAPE;
  return run(MORELLO_PATH_AUTO, 0, b, m, k, n, A, Bp, C, nullptr, 0, true, stream, true, strip);
}

#pragma GCC visibility pop
}  // extern "C"

namespace morello {
namespace {

// Float32 inputs: split into bf16 terms, then the bf16 problem (accumulating, or, `overwrite`,
// C = A x B with C never read).
int run_f32(int64_t b, int64_t m, int64_t k, int64_t n, const float* A, const float* B, float* C,
            void* stream, bool overwrite) {
  if (b < 0 || m < 0 || k < 0 || n < 0) return MORELLO_ERR_INVALID_SHAPE;
  int64_t k6, t;
  if (mul_overflows(k, 6, &k6) || mul_overflows(m, k6, &t) || mul_overflows(b, t, &t) ||
      mul_overflows(t, 2, &t) || mul_overflows(k6, n, &t) || mul_overflows(b, t, &t) ||
      mul_overflows(t, 2, &t))
    return MORELLO_ERR_INVALID_SHAPE;
  bool empty = false;
  // Shape, null and alignment checks of the bf16 problem the call turns into, with the
  // float pointers standing in (4-byte alignment is what they need).
  int rc = validate(b, m, k6, n, A, B, C, &empty);
  if (rc != MORELLO_OK) return rc;
  if (!empty && (reinterpret_cast<uintptr_t>(A) % 4 || reinterpret_cast<uintptr_t>(B) % 4))
    return MORELLO_ERR_MISALIGNED;
  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK) return rc;
  if (empty)   // an empty sum: the bf16 path knows what that means for either operation
    return run(MORELLO_PATH_AUTO, 0, b, m, k6, n, A, B, C, nullptr, 0, true, stream, overwrite);
  const size_t need = f32_split_bytes(b, m, k, n);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (st->split_bytes < need) {
      if (capturing(static_cast<cudaStream_t>(stream))) return MORELLO_ERR_WORKSPACE;
      cudaError_t e = cudaDeviceSynchronize();   // work in flight may still read the old buffer
      if (e != cudaSuccess) return cuda_fail(e);
      if (st->split) cudaFree(st->split);
      st->split = nullptr;
      st->split_bytes = 0;
      if ((e = cudaMalloc(&st->split, need)) != cudaSuccess) {
        cuda_fail(e);
        return MORELLO_ERR_WORKSPACE;
      }
      st->split_bytes = need;
    }
  }
  // When the bf16 problem goes to the tensor-core kernels directly and k is a whole number of
  // their 64-element blocks, only the three terms are stored and the kernels visit them in the
  // six-product order themselves (half the bytes written by the split); otherwise the six
  // products are laid out in full and any kernel can run the plain problem of 6k.
  const void* aligned = reinterpret_cast<const void*>(uintptr_t(4096));   // the split buffers are
  const bool three = k % 64 == 0 && !staged_wins(b, m, k6, n) &&
                     select_path(st->info.sms, b, m, k6, n, aligned, aligned, C) == MORELLO_PATH_TCGEN05;
  uint16_t *A6 = nullptr, *B6 = nullptr;
  uint64_t launches = 0;
  const cudaError_t e = f32_split_launch(b, m, k, n, A, B, st->split, !three, &A6, &B6,
                                         static_cast<cudaStream_t>(stream), &launches);
  g_launches.fetch_add(launches, std::memory_order_relaxed);
  if (e != cudaSuccess) return cuda_fail(e);
  if (!three) return run(MORELLO_PATH_AUTO, 0, b, m, k6, n, A6, B6, C, nullptr, 0, true, stream, overwrite);
  // Six segments of k / 64 blocks; stored terms 0, 1, 2 = first, second, third bf16 term.
  // A: 3, 1, 2, 2, 1, 1 and B: 1, 3, 2, 1, 2, 1 (smallest products first), three bits each.
  const KSegments seg{(int)(k / 64),
                      2u | (0u << 3) | (1u << 6) | (1u << 9) | (0u << 12) | (0u << 15),
                      0u | (2u << 3) | (1u << 6) | (0u << 9) | (1u << 12) | (0u << 15), 3 * k};
  return run(MORELLO_PATH_TCGEN05, 0, b, m, k6, n, A6, B6, C, nullptr, 0, true, stream, overwrite, 0, &seg);
}

}  // namespace
}  // namespace morello

#pragma GCC visibility push(default)
extern "C" {

int morello_matmul_accum_f32(int64_t b, int64_t m, int64_t k, int64_t n, const float* A,
                             const float* B, float* C, void* stream) {
  return run_f32(b, m, k, n, A, B, C, stream, false);
}

int morello_matmul_f32(int64_t b, int64_t m, int64_t k, int64_t n, const float* A, const float* B,
                       float* C, void* stream) {
  return run_f32(b, m, k, n, A, B, C, stream, true);
}

int morello_matmul_accum_host(int64_t b, int64_t m, int64_t k, int64_t n, const void* A_host,
                              const void* B_host, float* C_host) {
  bool empty = false;
  int rc = validate(b, m, k, n, A_host, B_host, C_host, &empty);
  if (rc != MORELLO_OK) return rc;
  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK || empty) return rc;
  auto round256 = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t a_bytes = (size_t)b * m * k * 2, b_bytes = (size_t)b * k * n * 2,
               c_bytes = (size_t)b * m * n * 4;
  const size_t need = round256(a_bytes) + round256(b_bytes) + round256(c_bytes);
  cudaError_t e;
  // One staging buffer per device: host threads take turns for the whole call (it is synchronous
  // anyway), so that neither the copies nor a regrowth of the buffer can cross another call.
  static std::mutex host_mutex;
  std::lock_guard<std::mutex> whole_call(host_mutex);
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (st->stage_bytes < need) {
      if ((e = cudaDeviceSynchronize()) != cudaSuccess) return cuda_fail(e);
      if (st->stage) cudaFree(st->stage);
      st->stage = nullptr;
      st->stage_bytes = 0;
      if ((e = cudaMalloc(&st->stage, need)) != cudaSuccess) {
        cuda_fail(e);
        return MORELLO_ERR_WORKSPACE;
      }
      st->stage_bytes = need;
    }
  }
  char* base = static_cast<char*>(st->stage);
  void* dA = base;
  void* dB = base + round256(a_bytes);
  float* dC = reinterpret_cast<float*>(base + round256(a_bytes) + round256(b_bytes));
  cudaStream_t s = cudaStreamPerThread;
  if ((e = cudaMemcpyAsync(dA, A_host, a_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
      (e = cudaMemcpyAsync(dB, B_host, b_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess ||
      (e = cudaMemcpyAsync(dC, C_host, c_bytes, cudaMemcpyHostToDevice, s)) != cudaSuccess)
    return cuda_fail(e);
  rc = run(MORELLO_PATH_AUTO, 0, b, m, k, n, dA, dB, dC, nullptr, 0, true, s);
  if (rc != MORELLO_OK) {
    cudaStreamSynchronize(s);
    return rc;
  }
  if ((e = cudaMemcpyAsync(C_host, dC, c_bytes, cudaMemcpyDeviceToHost, s)) != cudaSuccess ||
      (e = cudaStreamSynchronize(s)) != cudaSuccess)
    return cuda_fail(e);
  return MORELLO_OK;
}

int morello_select_path(int64_t b, int64_t m, int64_t k, int64_t n) {
  bool empty = false;
  const void* fake = reinterpret_cast<const void*>(uintptr_t(4096));
  if (validate(b, m, k, n, fake, fake, fake, &empty) != MORELLO_OK) return -1;
  // The choice depends on the SM count; without a usable device, a B200's is assumed.
  int sms = 148;
  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (device_state(&st) == MORELLO_OK) sms = st->info.sms;
  }
  if (!empty && staged_wins(b, m, k, n)) return MORELLO_PATH_TCGEN05;   // through padded copies
  return select_path(sms, b, m, k, n, fake, fake, fake);
}

int morello_describe_route(int64_t b, int64_t m, int64_t k, int64_t n, char* text, size_t text_bytes) {
  if (!text || text_bytes == 0) return MORELLO_ERR_NULL_POINTER;
  text[0] = 0;
  bool empty = false;
  const void* fake = reinterpret_cast<const void*>(uintptr_t(4096));   // 16-byte-aligned operands
  const int rc = validate(b, m, k, n, fake, fake, fake, &empty);
  if (rc != MORELLO_OK) return rc;
  if (empty) {
    snprintf(text, text_bytes, "nothing to launch (an empty sum)");
    return MORELLO_OK;
  }
  int sms = 148;   // without a usable device, a B200's
  DeviceState* st = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    if (device_state(&st) == MORELLO_OK) sms = st->info.sms;
  }
  TextOut out{text, text_bytes, 0};
#define put(...) out.append(__VA_ARGS__)
  int64_t kk = k, nn = n;
  const bool staged = staged_wins(b, m, k, n);
  if (staged) {
    const PadPlan pp = pad_plan(b, m, k, n, fake, fake, fake);
    kk = pp.k8;
    nn = pp.n8;
    put("padded copies of%s%s to k=%lld n=%lld%s, then ", pp.stage_a ? " A" : "", pp.stage_b ? " B" : "",
        (long long)kk, (long long)nn, pp.stage_c ? " (C written from registers)" : "");
  }
  const int path = staged ? MORELLO_PATH_TCGEN05 : select_path(sms, b, m, k, n, fake, fake, fake);
  if (path == MORELLO_PATH_TCGEN05) {
    const GemmPlan pl = gemm_plan(sms, b, m, kk, nn, 0);
    if (!pl.supported) return MORELLO_ERR_UNSUPPORTED_PATH;
    if (pl.form == 3) {
      put("tcgen05 swap_kernel: operands swapped, strips of 128 columns, %d rows of A per MMA", pl.tile_n);
      if (pl.split_k > 1) put(", %d k slices added inside a cluster", pl.split_k);
    } else {
      put("tcgen05 gemm_kernel: %s per %d x %d tile", pl.form == 2 ? "a CTA pair" : "one CTA",
          pl.form == 2 ? 256 : 128, pl.tile_n);
      const int64_t tile_m = pl.form == 2 ? 256 : 128;
      const int64_t tiles = b * ((m + tile_m - 1) / tile_m) * ((nn + pl.tile_n - 1) / pl.tile_n);
      const int64_t units = std::max(1, pl.form == 2 ? gemm_pair_units(sms) : sms);
      const int64_t tail = tiles % units;
      if (pl.halves && pl.ws_split <= 1 && (pl.tile_n / (pl.form == 2 ? 2 : 1) / 2) % 64 == 0 && tiles > units &&
          tail > 0 && 2 * tail <= units)
        put(", the %lld tiles of the last wave cut into column halves", (long long)tail);
    }
    if (pl.ws_split > 1) put(", %d k slices through the workspace + reduce launch", pl.ws_split);
  } else {
    const int which = skinny_kernel_for(0, b, m, k, n, fake);
    if (which == SKINNY_STREAM) {
      const StreamPlan pl = stream_plan(sms, b, (int)m, k, n, 0);
      put("fma gemv_stream_kernel: TMA ring, %d strips of 64 columns x %d k slices%s", pl.strips, pl.split_k,
          pl.split_k > 1 ? (pl.cluster_k ? " added inside a cluster" : " + reduce launch") : "");
    } else {
      const int rows = (int)std::min<int64_t>(kSkinnyMaxRows, m);
      const SkinnyPlan pl = skinny_plan(sms, b, rows, k, n, skinny_vec(n, fake), 0);
      put("fma skinny_kernel: register streaming%s, %lld chunk%s of <= 16 rows, %d-element loads, %d column blocks x %d k slices%s",
          pl.flat ? " (aligned granules, shifted columns)" : "", (long long)((m + kSkinnyMaxRows - 1) / kSkinnyMaxRows),
          m > kSkinnyMaxRows ? "s" : "", pl.vec, pl.col_blocks, pl.split_k, pl.split_k > 1 ? " + reduce launch" : "");
    }
  }
#undef put
  return MORELLO_OK;
}

int morello_read_device_status(void* stream, uint32_t* detail) {
  if (detail) *detail = 0;
  DeviceState* st = nullptr;
  int rc;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e);
  uint32_t word = 0;
  if ((e = cudaMemcpy(&word, st->info.status, 4, cudaMemcpyDeviceToHost)) != cudaSuccess)
    return cuda_fail(e);
  if (word == 0) return MORELLO_OK;
  if ((e = cudaMemset(st->info.status, 0, 4)) != cudaSuccess) return cuda_fail(e);
  if (detail) *detail = word;
  return MORELLO_ERR_DEVICE_TIMEOUT;
}

int morello_selftest_wait_timeout(uint32_t limit_ms, void* stream) {
  if (limit_ms == 0 || limit_ms > 1000) return MORELLO_ERR_INVALID_SHAPE;
  DeviceState* st = nullptr;
  int rc;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK) return rc;
  // The second word of the status block receives the kernel's own verdict.
  int* gave_up = reinterpret_cast<int*>(st->info.status + 1);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(gave_up, 0, 4, s);
  if (e != cudaSuccess) return cuda_fail(e);
  e = wait_timeout_selftest_launch(st->info.status, (uint64_t)limit_ms * 1000000ull, gave_up, s);
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if ((e = cudaStreamSynchronize(s)) != cudaSuccess) return cuda_fail(e);
  int verdict = 0;
  if ((e = cudaMemcpy(&verdict, gave_up, 4, cudaMemcpyDeviceToHost)) != cudaSuccess) return cuda_fail(e);
  return verdict == 1 ? MORELLO_OK : MORELLO_ERR_CUDA;
}

int morello_selftest_per_device_once(int devices, int calls_per_device) {
  if (devices < 0 || calls_per_device < 0) return -1;
  PerDeviceOnce once;
  int runs = 0;
  for (int c = 0; c < calls_per_device; ++c)
    for (int d = 0; d < devices; ++d)
      // A first attempt that fails is not remembered: device 1's set-up fails once, then works.
      (void)once.run(d, [&] {
        ++runs;
        return (d == 1 && runs <= devices) ? cudaErrorInvalidValue : cudaSuccess;
      });
  return runs;
}

int morello_device_limits(int* sms, int* cta_pairs) {
  DeviceState* st = nullptr;
  int rc;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    rc = device_state(&st);
  }
  if (rc != MORELLO_OK) return rc;
  if (sms) *sms = st->info.sms;
  if (cta_pairs) *cta_pairs = gemm_pair_units(st->info.sms);
  return MORELLO_OK;
}

uint64_t morello_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int morello_last_cuda_error(void) { return t_last_cuda_error; }

const char* morello_status_string(int status) {
  switch (status) {
    case MORELLO_OK: return "ok";
    case MORELLO_ERR_INVALID_SHAPE: return "invalid shape (negative dimension or size overflow)";
    case MORELLO_ERR_NULL_POINTER: return "null pointer for a non-empty tensor";
    case MORELLO_ERR_MISALIGNED: return "pointer not aligned to its element type (or workspace to 16 bytes)";
    case MORELLO_ERR_UNSUPPORTED_DEVICE: return "current device is not compute capability 10.x";
    case MORELLO_ERR_WORKSPACE: return "workspace too small or its allocation failed";
    case MORELLO_ERR_CUDA: return "a CUDA call failed (see morello_last_cuda_error)";
    case MORELLO_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
    case MORELLO_ERR_UNSUPPORTED_PATH: return "the forced path cannot run this shape or alignment";
    default: return "unknown status";
  }
}

const char* morello_version(void) { return "morello-b200 0.1 (sm_100a)"; }

}  // extern "C"
#pragma GCC visibility pop
