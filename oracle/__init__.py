"""CPU oracle for MatmulAccum -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin ctypes loader around ``morello_oracle.c`` (plain C, double accumulation,
one rounding to f32; see that file's header for the passages of the paper it
follows).  Only the tests, the smoke check and the benchmark's CPU-baseline /
reference leg may import this package.  It imports nothing from the CUDA
package and the CUDA package imports nothing from here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "morello_oracle.c")
_LIB = os.path.join(_HERE, "libmorello_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP for the row-parallel loops)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp",
           "-ffp-contract=off", "-fno-fast-math", "-Wall", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, vp = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_matmul_accum_naive.argtypes = [i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_matmul_accum_naive.restype = None
        lib.oracle_matmul_accum.argtypes = [i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_matmul_accum.restype = ctypes.c_int
        lib.oracle_matmul_accum_rows.argtypes = [i64, i64, i64, i64, vp, vp, vp,
                                                 i64, vp, vp, vp]
        lib.oracle_matmul_accum_rows.restype = ctypes.c_int
        lib.oracle_abs_dot.argtypes = [i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_abs_dot.restype = None
        lib.oracle_matmul_accum_f32.argtypes = [i64, i64, i64, i64, vp, vp, vp, vp]
        lib.oracle_matmul_accum_f32.restype = ctypes.c_int
        lib.oracle_matmul_accum_bt.argtypes = [i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_matmul_accum_bt.restype = None
        lib.oracle_matmul_accum_packed_b.argtypes = [i64, i64, i64, i64, i64, vp, vp, vp]
        lib.oracle_matmul_accum_packed_b.restype = None
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _check(A, B, C, b, m, k, n):
    assert A.dtype == np.uint16 and A.flags.c_contiguous and A.size == b * m * k
    assert B.dtype == np.uint16 and B.flags.c_contiguous and B.size == b * k * n
    assert C.dtype == np.float32 and C.flags.c_contiguous and C.size == b * m * n


def _ptr(x):
    return x.ctypes.data if x is not None and x.size else None


def matmul_accum(b, m, k, n, A, B, C, naive: bool = False) -> np.ndarray:
    """Return C + A x B (new f32 array); A, B are bf16 bit patterns (uint16)."""
    _check(A, B, C, b, m, k, n)
    out = np.array(C, dtype=np.float32, copy=True, order="C")
    lib = _load()
    if naive:
        lib.oracle_matmul_accum_naive(b, m, k, n, _ptr(A), _ptr(B), _ptr(out))
    else:
        rc = lib.oracle_matmul_accum(b, m, k, n, _ptr(A), _ptr(B), _ptr(out))
        if rc != 0:
            raise MemoryError("oracle scratch allocation failed")
    return out


def matmul_accum_rows(b, m, k, n, A, B, C, rows, want_abs: bool = True):
    """Oracle result for the flattened rows ``bb*m + i`` in ``rows``.

    Returns (out[nrows, n] f32, T[nrows, n] f64 or None)."""
    _check(A, B, C, b, m, k, n)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < b * m)
    out = np.zeros((rows.size, n), dtype=np.float32)
    T = np.zeros((rows.size, n), dtype=np.float64) if want_abs else None
    rc = _load().oracle_matmul_accum_rows(b, m, k, n, _ptr(A), _ptr(B), _ptr(C),
                                          rows.size, _ptr(rows), _ptr(out), _ptr(T))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return out, T


def abs_dot(b, m, k, n, A, B) -> np.ndarray:
    """T[b,i,j] = sum_p |A*B| in f64, shape (b, m, n)."""
    assert A.dtype == np.uint16 and B.dtype == np.uint16
    T = np.zeros((b, m, n), dtype=np.float64)
    _load().oracle_abs_dot(b, m, k, n, _ptr(A), _ptr(B), _ptr(T))
    return T


def matmul_accum_f32(b, m, k, n, A, B, C, want_abs: bool = False):
    """float32 inputs: returns C + A x B (new f32 array), and sum_p |A*B| (f64) if asked."""
    for x, size in ((A, b * m * k), (B, b * k * n), (C, b * m * n)):
        assert x.dtype == np.float32 and x.flags.c_contiguous and x.size == size
    out = np.array(C, dtype=np.float32, copy=True, order="C")
    T = np.zeros((b, m, n), dtype=np.float64) if want_abs else None
    rc = _load().oracle_matmul_accum_f32(b, m, k, n, _ptr(A), _ptr(B), _ptr(out), _ptr(T))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return (out, T) if want_abs else out


def matmul_accum_bt(b, m, k, n, A, Bt, C) -> np.ndarray:
    """B given column-major (Bt[b][n][k], bf16 bit patterns): returns C + A x B."""
    assert Bt.dtype == np.uint16 and Bt.flags.c_contiguous and Bt.size == b * n * k
    assert A.dtype == np.uint16 and A.flags.c_contiguous and A.size == b * m * k
    out = np.array(C, dtype=np.float32, copy=True, order="C")
    assert out.size == b * m * n
    _load().oracle_matmul_accum_bt(b, m, k, n, _ptr(A), _ptr(Bt), _ptr(out))
    return out


def matmul_accum_packed_b(strip, b, m, k, n, A, Bp, C) -> np.ndarray:
    """B given packed in strips of `strip` columns (Bp[b][ceil(n/strip)][k][strip], bf16 bit
    patterns, last strip padded): returns C + A x B."""
    strips = (n + strip - 1) // strip
    assert Bp.dtype == np.uint16 and Bp.flags.c_contiguous and Bp.size == b * strips * k * strip
    assert A.dtype == np.uint16 and A.flags.c_contiguous and A.size == b * m * k
    out = np.array(C, dtype=np.float32, copy=True, order="C")
    assert out.size == b * m * n
    _load().oracle_matmul_accum_packed_b(strip, b, m, k, n, _ptr(A), _ptr(Bp), _ptr(out))
    return out


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(t: int) -> None:
    _load().oracle_set_num_threads(int(t))
