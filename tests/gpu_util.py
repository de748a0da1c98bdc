"""Helpers for the GPU parity tests: move seeded inputs to the device, call the
library through its C ABI binding, and compare with the CPU oracle under the
acceptance rule (bit-exact on integer inputs, else
|gpu - oracle| <= 1e-5 * sum_p |A*B| + 1e-6)."""
import numpy as np
import torch

import oracle
from paper_2505_01637_b200 import binding as mb

RTOL_ABS_DOT = 1e-5
ATOL = 1e-6


def to_dev(A, B, C):
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = torch.from_numpy(B.view(np.int16)).cuda()
    dC = torch.from_numpy(C.copy()).cuda()
    return dA, dB, dC


def gpu_run(A, B, C, path=mb.MORELLO_PATH_AUTO, split_k=0, calls=1):
    b, m, k = A.shape
    n = B.shape[2]
    dA, dB, dC = to_dev(A, B, C)
    for _ in range(calls):
        if path == mb.MORELLO_PATH_AUTO and split_k == 0:
            mb.morello_matmul_accum(b, m, k, n, dA, dB, dC)
        else:
            mb.morello_matmul_accum_forced(path, split_k, b, m, k, n, dA, dB, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, "device status %d detail 0x%x" % (st, detail)
    return dC.cpu().numpy()


def bits(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


def assert_bit_exact(got, want, what=""):
    if not np.array_equal(bits(got), bits(want)):
        bad = np.argwhere(bits(got) != bits(want))
        first = tuple(bad[0])
        raise AssertionError("%s: %d of %d elements differ; first at %s: got %r want %r" % (
            what, len(bad), got.size, first, got[first], want[first]))


def assert_within_tolerance(got, want, T, what=""):
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = RTOL_ABS_DOT * T + ATOL
    ratio = float((err / bound).max()) if err.size else 0.0
    assert ratio <= 1.0, "%s: max |gpu-oracle| / (1e-5*T+1e-6) = %.3f" % (what, ratio)
    return ratio


def check_full(A, B, C, integer, path=mb.MORELLO_PATH_AUTO, split_k=0, what=""):
    """Whole-output comparison against the oracle."""
    b, m, k = A.shape
    n = B.shape[2]
    got = gpu_run(A, B, C, path, split_k)
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    if integer:
        assert_bit_exact(got, want, what)
    else:
        assert_within_tolerance(got, want, oracle.abs_dot(b, m, k, n, A, B), what)
    return got


def check_rows(A, B, C, rows, integer, got, what=""):
    """Comparison of sampled rows (flattened ids bb*m + i) against the oracle."""
    b, m, k = A.shape
    n = B.shape[2]
    want, T = oracle.matmul_accum_rows(b, m, k, n, A, B, C, rows, want_abs=not integer)
    sub = got.reshape(b * m, n)[rows]
    if integer:
        assert_bit_exact(sub, want, what)
    else:
        assert_within_tolerance(sub, want, T, what)
