"""MatmulAccum with B packed in strips of columns (Section 2.4.2 of the paper) against the CPU
oracle: the tensor-core kernels for strips that are multiples of 64 columns, the plain kernel
for everything else."""
import numpy as np
import pytest

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance, bits, to_dev

pytestmark = pytest.mark.gpu
NAN = 0x7FC0      # padding of the last strip: must never reach a result


def _run(strip, A, B, C, calls=1):
    b, m, k = A.shape
    n = B.shape[2]
    Bp = w.pack_b(B, strip, fill=NAN)
    dA, dBp, dC = to_dev(A, Bp, C)
    for _ in range(calls):
        mb.morello_matmul_accum_packed_b(strip, b, m, k, n, dA, dBp, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    return dC.cpu().numpy(), Bp


@pytest.mark.parametrize("strip", [64, 128, 256])
@pytest.mark.parametrize("shape", [
    (1, 128, 64, 256),       # one tile
    (1, 1, 2048, 4096),      # one row: the operand-swapped kernel
    (2, 16, 520, 776),       # few rows, ragged k and n (last strip padded)
    (1, 300, 1000, 328),     # ragged tiles
    (3, 64, 136, 200),
    (1, 8, 4096, 256),       # few strips, long k: k slices inside a cluster
    (1, 512, 8192, 264),     # few tiles, long k: k slices through the workspace
    (1, 2048, 128, 2056),    # many tiles, a column tile past the last strip
])
def test_packed_b_on_the_tensor_kernels(shape, strip):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + strip, ab="int4", c="normal")
    got, Bp = _run(strip, A, B, C)
    assert_bit_exact(got, oracle.matmul_accum_packed_b(strip, b, m, k, n, A, Bp.reshape(-1), C), "packed %d %s" % (strip, shape))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + strip + 1, ab="normal_rsqrtk", c="normal")
    got, Bp = _run(strip, A, B, C)
    want = oracle.matmul_accum_packed_b(strip, b, m, k, n, A, Bp.reshape(-1), C)
    assert_within_tolerance(got, want, oracle.abs_dot(b, m, k, n, A, B), "packed %d %s random" % (strip, shape))
    again, _ = _run(strip, A, B, C)
    assert np.array_equal(bits(again), bits(got))


@pytest.mark.parametrize("strip,shape", [
    (8, (2, 5, 33, 50)),       # the strip of a vector register: plain kernel
    (16, (1, 40, 100, 72)),
    (64, (1, 17, 63, 130)),    # k % 8 != 0: plain kernel although the strip would do
    (4, (1, 3, 7, 9)),
    (1, (2, 4, 24, 16)),       # strip 1 = column-major
    (100, (1, 9, 16, 250)),
])
def test_packed_b_on_the_plain_kernel(strip, shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + strip, ab="int4", c="normal")
    got, Bp = _run(strip, A, B, C)
    assert_bit_exact(got, oracle.matmul_accum_packed_b(strip, b, m, k, n, A, Bp.reshape(-1), C), "packed %d %s" % (strip, shape))
    twice, _ = _run(strip, A, B, C, calls=2)
    want2 = oracle.matmul_accum_packed_b(strip, b, m, k, n, A, Bp.reshape(-1),
                                         oracle.matmul_accum_packed_b(strip, b, m, k, n, A, Bp.reshape(-1), C))
    assert_bit_exact(twice, want2, "two accumulating calls")


def test_packed_b_one_hot_pins_the_strip_arithmetic():
    strip, b, m, k, n = 64, 2, 20, 136, 200          # 4 strips per batch, the last 8 columns wide
    rng = np.random.default_rng(3)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, p0, j0) in [(0, 0, 0), (0, 70, 63), (0, 70, 64), (1, 135, 199), (1, 64, 128)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[b0, p0, j0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        got, _ = _run(strip, w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C)
        assert_bit_exact(got, want, "one-hot B at %s" % ((b0, p0, j0),))


def test_packed_b_bad_strip_and_empty_shapes():
    import torch
    d = torch.zeros(64, dtype=torch.int16, device="cuda")
    c = torch.full((2, 8), 3.0, device="cuda")
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_packed_b(0, 1, 2, 4, 8, d, d, c)
    assert e.value.status == mb.MORELLO_ERR_INVALID_SHAPE
    mb.morello_matmul_accum_packed_b(64, 1, 2, 0, 8, d, d, c)     # empty sum: C untouched
    torch.cuda.synchronize()
    assert float(c.min()) == 3.0 and float(c.max()) == 3.0


@pytest.mark.parametrize("shape", [(1, 16, 520, 776), (2, 300, 1000, 328), (1, 5, 33, 50), (1, 8, 4096, 256)])
def test_matmul_with_b_column_major_or_packed_never_reads_c(shape):
    import torch
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    want = oracle.matmul_accum(b, m, k, n, A, B, np.zeros_like(C))
    poison = np.full_like(C, np.nan)
    dA, dBp, dC = to_dev(A, w.pack_b(B, 64, fill=NAN), poison)
    mb.morello_matmul_packed_b(64, b, m, k, n, dA, dBp, dC)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), want, "matmul, packed B %s" % (shape,))
    dA, dBt, dC = to_dev(A, np.ascontiguousarray(np.swapaxes(B, 1, 2)), poison)
    mb.morello_matmul_colmajor_b(0, b, m, k, n, dA, dBt, dC)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), want, "matmul, column-major B %s" % (shape,))
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
