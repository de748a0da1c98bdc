"""Python binding of the C ABI (``include/morello.h``): argument marshalling only.

Every function has the name and argument order of its C counterpart.  Tensor
arguments may be torch CUDA tensors (their ``data_ptr()`` is passed) or plain
integer device addresses; ``stream`` may be a ``torch.cuda.Stream``, an integer
``cudaStream_t`` or None (torch's current stream when torch is loaded and CUDA is
up, else the default stream).  Status codes other than MORELLO_OK raise
``MorelloError``.  There is no fallback: if the shared library has not been
built, importing this module's functions raises."""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmorello.so")

MORELLO_OK = 0
MORELLO_ERR_INVALID_SHAPE = 1
MORELLO_ERR_NULL_POINTER = 2
MORELLO_ERR_MISALIGNED = 3
MORELLO_ERR_UNSUPPORTED_DEVICE = 4
MORELLO_ERR_WORKSPACE = 5
MORELLO_ERR_CUDA = 6
MORELLO_ERR_DEVICE_TIMEOUT = 7
MORELLO_ERR_UNSUPPORTED_PATH = 8

MORELLO_PATH_AUTO = -1
MORELLO_PATH_SKINNY = 0
MORELLO_PATH_TCGEN05 = 1

_i64, _vp, _int, _sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/morello.h declaration by declaration
SIGNATURES = {
    "morello_matmul_accum": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul_forced": (_int, [_int, _int, _i64, _i64, _i64, _i64, _vp, _vp, _vp,
                                     _vp, _sz, _vp]),
    "morello_matmul_accum_f32": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul_f32": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul_accum_colmajor_b": (_int, [_int, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul_accum_packed_b": (_int, [_int, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_selftest_wait_timeout": (_int, [ctypes.c_uint32, _vp]),
    "morello_matmul_colmajor_b": (_int, [_int, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_matmul_packed_b": (_int, [_int, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_workspace_bytes": (_sz, [_i64, _i64, _i64, _i64]),
    "morello_matmul_accum_ws": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp, _sz, _vp]),
    "morello_matmul_accum_host": (_int, [_i64, _i64, _i64, _i64, _vp, _vp, _vp]),
    "morello_matmul_accum_noalloc": (_int, [_int, _i64, _i64, _i64, _i64, _vp, _vp, _vp, _vp]),
    "morello_noalloc_scratch_limit": (_sz, []),
    "morello_select_path": (_int, [_i64, _i64, _i64, _i64]),
    "morello_describe_route": (_int, [_i64, _i64, _i64, _i64, ctypes.c_char_p, _sz]),
    "morello_selftest_per_device_once": (_int, [_int, _int]),
    "morello_matmul_accum_forced": (_int, [_int, _int, _i64, _i64, _i64, _i64, _vp, _vp, _vp,
                                           _vp, _sz, _vp]),
    "morello_workspace_bytes_forced": (_sz, [_int, _int, _i64, _i64, _i64, _i64]),
    "morello_read_device_status": (_int, [_vp, ctypes.POINTER(ctypes.c_uint32)]),
    "morello_device_limits": (_int, [ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int)]),
    "morello_launch_count": (ctypes.c_uint64, []),
    "morello_last_cuda_error": (_int, []),
    "morello_status_string": (ctypes.c_char_p, [_int]),
    "morello_version": (ctypes.c_char_p, []),
}


class MorelloError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = lib().morello_status_string(self.status).decode()
        if self.status == MORELLO_ERR_CUDA:
            msg += " [cudaError %d]" % lib().morello_last_cuda_error()
        super().__init__("%s: %s (status %d)" % (where, msg, self.status))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "%s is missing: build it with `python -m paper_2505_01637_b200.build` "
                "(there is no fallback implementation)" % LIB_PATH)
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _addr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x or None
    if hasattr(x, "data_ptr"):
        return x.data_ptr() or None
    if hasattr(x, "ctypes"):          # numpy array (host entry point)
        return x.ctypes.data or None
    raise TypeError("expected a tensor, an array or an integer address, got %r" % type(x))


def _stream(stream):
    if stream is None:
        import sys
        torch = sys.modules.get("torch")
        if torch is not None and torch.cuda.is_available():
            return torch.cuda.current_stream().cuda_stream or None
        return None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(status: int, where: str) -> None:
    if status != MORELLO_OK:
        raise MorelloError(status, where)


def morello_matmul_accum(b, m, k, n, A, B, C, stream=None) -> None:
    _check(lib().morello_matmul_accum(b, m, k, n, _addr(A), _addr(B), _addr(C), _stream(stream)),
           "morello_matmul_accum")


def morello_matmul(b, m, k, n, A, B, C, stream=None) -> None:
    """C = A x B (C's prior contents are not read)."""
    _check(lib().morello_matmul(b, m, k, n, _addr(A), _addr(B), _addr(C), _stream(stream)),
           "morello_matmul")


def morello_matmul_forced(path, split_k, b, m, k, n, A, B, C, workspace=None,
                          workspace_bytes=0, stream=None) -> None:
    _check(lib().morello_matmul_forced(path, split_k, b, m, k, n, _addr(A), _addr(B), _addr(C),
                                       _addr(workspace), workspace_bytes, _stream(stream)),
           "morello_matmul_forced")


def morello_matmul_accum_f32(b, m, k, n, A, B, C, stream=None) -> None:
    """C += A x B with float32 A and B (split into bf16 terms inside the library)."""
    _check(lib().morello_matmul_accum_f32(b, m, k, n, _addr(A), _addr(B), _addr(C), _stream(stream)),
           "morello_matmul_accum_f32")


def morello_matmul_f32(b, m, k, n, A, B, C, stream=None) -> None:
    """C = A x B with float32 A and B (C is not read)."""
    _check(lib().morello_matmul_f32(b, m, k, n, _addr(A), _addr(B), _addr(C), _stream(stream)),
           "morello_matmul_f32")


def morello_matmul_accum_colmajor_b(tile, b, m, k, n, A, Bt, C, stream=None) -> None:
    """C += A x B with B given column-major: Bt[b][n][k]."""
    _check(lib().morello_matmul_accum_colmajor_b(tile, b, m, k, n, _addr(A), _addr(Bt), _addr(C),
                                                 _stream(stream)),
           "morello_matmul_accum_colmajor_b")


def morello_matmul_accum_packed_b(strip, b, m, k, n, A, Bp, C, stream=None) -> None:
    """C += A x B with B packed in strips of `strip` columns: Bp[b][ceil(n/strip)][k][strip]."""
    _check(lib().morello_matmul_accum_packed_b(strip, b, m, k, n, _addr(A), _addr(Bp), _addr(C),
                                               _stream(stream)),
           "morello_matmul_accum_packed_b")


def morello_matmul_colmajor_b(tile, b, m, k, n, A, Bt, C, stream=None) -> None:
    """C = A x B with B given column-major (C is not read)."""
    _check(lib().morello_matmul_colmajor_b(tile, b, m, k, n, _addr(A), _addr(Bt), _addr(C), _stream(stream)),
           "morello_matmul_colmajor_b")


def morello_matmul_packed_b(strip, b, m, k, n, A, Bp, C, stream=None) -> None:
    """C = A x B with B packed in strips of `strip` columns (C is not read)."""
    _check(lib().morello_matmul_packed_b(strip, b, m, k, n, _addr(A), _addr(Bp), _addr(C), _stream(stream)),
           "morello_matmul_packed_b")


def morello_workspace_bytes(b, m, k, n) -> int:
    return int(lib().morello_workspace_bytes(b, m, k, n))


def morello_matmul_accum_ws(b, m, k, n, A, B, C, workspace, workspace_bytes, stream=None) -> None:
    _check(lib().morello_matmul_accum_ws(b, m, k, n, _addr(A), _addr(B), _addr(C),
                                         _addr(workspace), workspace_bytes, _stream(stream)),
           "morello_matmul_accum_ws")


def morello_matmul_accum_host(b, m, k, n, A_host, B_host, C_host) -> None:
    _check(lib().morello_matmul_accum_host(b, m, k, n, _addr(A_host), _addr(B_host), _addr(C_host)),
           "morello_matmul_accum_host")


def morello_matmul_accum_noalloc(split_k, b, m, k, n, A, B, C, stream=None) -> None:
    """Allocation-free variant: partial sums live in a fixed array inside the library."""
    _check(lib().morello_matmul_accum_noalloc(split_k, b, m, k, n, _addr(A), _addr(B), _addr(C),
                                              _stream(stream)),
           "morello_matmul_accum_noalloc")


def morello_noalloc_scratch_limit() -> int:
    return int(lib().morello_noalloc_scratch_limit())


def morello_select_path(b, m, k, n) -> int:
    return int(lib().morello_select_path(b, m, k, n))


def morello_describe_route(b, m, k, n) -> str:
    """One line naming the kernel, tile and k slices the selector picks for this shape."""
    buf = ctypes.create_string_buffer(512)
    _check(lib().morello_describe_route(b, m, k, n, buf, len(buf)), "morello_describe_route")
    return buf.value.decode()


def morello_selftest_per_device_once(devices, calls_per_device) -> int:
    return int(lib().morello_selftest_per_device_once(devices, calls_per_device))


def morello_matmul_accum_forced(path, split_k, b, m, k, n, A, B, C, workspace=None,
                                workspace_bytes=0, stream=None) -> None:
    _check(lib().morello_matmul_accum_forced(path, split_k, b, m, k, n, _addr(A), _addr(B),
                                             _addr(C), _addr(workspace), workspace_bytes,
                                             _stream(stream)),
           "morello_matmul_accum_forced")


def morello_workspace_bytes_forced(path, split_k, b, m, k, n) -> int:
    return int(lib().morello_workspace_bytes_forced(path, split_k, b, m, k, n))


def morello_selftest_wait_timeout(limit_ms, stream=None) -> None:
    """Makes one bounded device-side wait run out on purpose (see the header); raises unless it
    gave up as designed.  The device status word is set afterwards."""
    _check(lib().morello_selftest_wait_timeout(limit_ms, _stream(stream)), "morello_selftest_wait_timeout")


def morello_read_device_status(stream=None):
    """Returns (status, detail) after synchronising the stream; does not raise."""
    detail = ctypes.c_uint32(0)
    st = lib().morello_read_device_status(_stream(stream), ctypes.byref(detail))
    return int(st), int(detail.value)


def morello_device_limits():
    """(SMs, two-CTA clusters the device holds at once) of the current device."""
    sms, pairs = ctypes.c_int(0), ctypes.c_int(0)
    _check(lib().morello_device_limits(ctypes.byref(sms), ctypes.byref(pairs)), "morello_device_limits")
    return int(sms.value), int(pairs.value)


def morello_launch_count() -> int:
    return int(lib().morello_launch_count())


def morello_last_cuda_error() -> int:
    return int(lib().morello_last_cuda_error())


def morello_status_string(status: int) -> str:
    return lib().morello_status_string(int(status)).decode()


def morello_version() -> str:
    return lib().morello_version().decode()
