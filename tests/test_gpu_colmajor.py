"""GPU parity of MatmulAccum with a column-major right-hand side (Bt[b][n][k]) against the
CPU oracle for that layout: every tensor-core form, the plain kernel for shapes the TMA
engine cannot address, operand-layout pins."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance

pytestmark = pytest.mark.gpu


def _run(shape, A, Bt, C, tile=0, calls=1):
    b, m, k, n = shape
    dA = torch.from_numpy(A.view(np.int16)).cuda()
    dB = torch.from_numpy(Bt.view(np.int16)).cuda()
    dC = torch.from_numpy(C.copy()).cuda()
    for _ in range(calls):
        mb.morello_matmul_accum_colmajor_b(tile, b, m, k, n, dA, dB, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    return dC.cpu().numpy()


CASES = [
    (0, (1, 4, 128, 16)),        # the Spec example's shape
    (0, (1, 1, 2048, 16384)),    # the GEMV with column-major weights
    (0, (1, 16, 2048, 4096)),
    (3, (2, 5, 200, 264)),       # operand-swapped kernel, ragged
    (3, (1, 33, 72, 136)),
    (3 + 16 * 8, (1, 16, 4096, 264)),   # ... eight k slices in a cluster
    (1, (1, 100, 72, 200)),      # one-CTA tiles, ragged
    (16 + 1, (1, 200, 136, 72)),
    (2, (2, 300, 520, 776)),     # CTA-pair tiles, ragged
    (32 + 2, (1, 512, 256, 384)),
    (64 + 2, (2, 1100, 72, 4504)),   # last wave cut into halves
    (0, (2, 3, 50, 24)),         # k % 8 != 0: the one-warp-per-column kernel
    (0, (1, 40, 64, 36)),        # n % 8 != 0: likewise
]


@pytest.mark.parametrize("tile,shape", CASES)
def test_colmajor_b_matches_oracle(tile, shape):
    b, m, k, n = shape
    for dist, integer in (("int4", True), ("uniform", False)):
        A, B, C = w.make(b, m, k, n, seed=sum(shape) + tile, ab=dist, c="normal")
        Bt = np.ascontiguousarray(B.transpose(0, 2, 1))
        want = oracle.matmul_accum_bt(b, m, k, n, A, Bt, C)
        got = _run(shape, A, Bt, C, tile)
        if integer:
            assert_bit_exact(got, want, "col-major B %s tile %d" % (shape, tile))
        else:
            assert_within_tolerance(got, want, oracle.abs_dot(b, m, k, n, A, B), "col-major B %s" % (shape,))


@pytest.mark.parametrize("tile", [0, 1, 2, 3])
def test_colmajor_b_one_hot_operands(tile):
    b, m, k, n = 2, 40, 136, 328
    rng = np.random.default_rng(tile)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    Btv = rng.integers(-100, 101, size=(b, n, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, i0, p0) in [(0, 0, 0), (1, 39, 135), (1, 17, 64)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Btv[b0, :, p0]
        got = _run((b, m, k, n), w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Btv), C, tile)
        assert_bit_exact(got, want, "one-hot A at %s" % ((b0, i0, p0),))
    for (b0, j0, p0) in [(0, 0, 0), (1, 327, 135), (1, 128, 64)]:
        B1 = np.zeros((b, n, k), np.float32)
        B1[b0, j0, p0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        got = _run((b, m, k, n), w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C, tile)
        assert_bit_exact(got, want, "one-hot Bt at %s" % ((b0, j0, p0),))


def test_colmajor_b_accumulates_and_repeats():
    shape = (1, 192, 256, 384)
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=3, ab="int4", c="int8")
    Bt = np.ascontiguousarray(B.transpose(0, 2, 1))
    twice = oracle.matmul_accum_bt(b, m, k, n, A, Bt, oracle.matmul_accum_bt(b, m, k, n, A, Bt, C))
    assert_bit_exact(_run(shape, A, Bt, C, calls=2), twice, "two accumulating calls")
    A, B, C = w.make(b, m, k, n, seed=4, ab="normal_rsqrtk", c="normal")
    Bt = np.ascontiguousarray(B.transpose(0, 2, 1))
    first = _run(shape, A, Bt, C)
    assert np.array_equal(_run(shape, A, Bt, C).view(np.uint32), first.view(np.uint32))
