"""The register-streaming kernel's flat form: a B whose rows are not 16-byte aligned (n % 8 != 0,
or a base that is not 16-byte aligned) is read in aligned 16-byte granules, every row lane's
accumulators standing for columns shifted by that lane's offset inside the granule.  Parity
with the CPU oracle, bit-exact on integer inputs; every offset 0..7 and both parities of n
occur among the cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, bits, check_full, gpu_run, to_dev

pytestmark = pytest.mark.gpu
SK = mb.MORELLO_PATH_SKINNY
REG = 1024            # knob: the register-streaming kernel


@pytest.mark.parametrize("shape", [
    (1, 1, 2048, 16383),    # the headline shape less one column: n odd, every offset occurs
    (1, 1, 768, 50257),     # an odd vocabulary size
    (1, 1, 1000, 1001),     # ragged k
    (1, 2, 515, 770),       # n % 8 == 2
    (1, 3, 4096, 516),      # n % 8 == 4; few columns: k slices through scratch
    (2, 4, 520, 777),       # batches, 4 rows
    (3, 1, 129, 70),        # a last block of 6 columns; granules reach the end of B
    (1, 1, 128, 63),
    (1, 8, 300, 262),
    (1, 16, 200, 1027),
    (2, 20, 100, 519),      # two row chunks
    (1, 1, 16384, 2054),    # long k
    (1, 5, 64, 17),         # the smallest shape that takes this form
])
def test_flat_form_matches_the_oracle(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    check_full(A, B, C, integer=True, path=SK, split_k=REG, what="flat %s" % (shape,))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="uniform_rsqrtk", c="normal")
    first = check_full(A, B, C, integer=False, path=SK, split_k=REG, what="flat %s random" % (shape,))
    assert np.array_equal(bits(gpu_run(A, B, C, path=SK, split_k=REG)), bits(first))


@pytest.mark.parametrize("split", [2, 3, 7])
def test_flat_form_with_forced_k_slices(split):
    b, m, k, n = 2, 3, 1000, 333
    A, B, C = w.make(b, m, k, n, seed=split, ab="int4", c="normal")
    whole = check_full(A, B, C, integer=True, path=SK, split_k=REG + 1, what="one slice")
    assert_bit_exact(gpu_run(A, B, C, path=SK, split_k=REG + split), whole, "%d slices" % split)


@pytest.mark.parametrize("off", [1, 2, 3, 5, 7])
def test_flat_form_with_b_at_odd_addresses(off):
    # n % 8 == 0 but B starts `off` elements past a 16-byte boundary.
    b, m, k, n = 2, 2, 700, 512
    A, B, C = w.make(b, m, k, n, seed=off, ab="int4", c="normal")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    buf = torch.zeros(B.size + 16, dtype=torch.int16, device="cuda")
    dB = buf[off:off + B.size]
    dB.copy_(torch.from_numpy(B.view(np.int16).reshape(-1)))
    assert dB.data_ptr() % 16 == 2 * off
    dA, _, dC = to_dev(A, B, C)
    mb.morello_matmul_accum(b, m, k, n, dA, dB.data_ptr(), dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    assert_bit_exact(dC.cpu().numpy(), want, "B %d elements off" % off)


def test_flat_form_one_hot_rows_and_columns():
    b, m, k, n = 1, 2, 300, 333
    rng = np.random.default_rng(4)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (i0, p0) in [(0, 0), (1, 299), (0, 128), (1, 7)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[0, i0, p0] = 2.0
        want = C.copy()
        want[0, i0, :] += 2.0 * Bv[0, p0, :]
        got = gpu_run(w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Bv), C, path=SK, split_k=REG)
        assert_bit_exact(got, want, "one-hot A at %s" % ((i0, p0),))
    for (p0, j0) in [(0, 0), (299, 332), (130, 64), (5, 63), (77, 200), (8, 128), (9, 127)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[0, p0, j0] = -3.0
        want = C.copy()
        want[0, :, j0] += -3.0 * Av[0, :, p0]
        got = gpu_run(w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C, path=SK, split_k=REG)
        assert_bit_exact(got, want, "one-hot B at %s" % ((p0, j0),))


def test_selector_reaches_the_flat_form():
    for shape in [(1, 1, 2048, 16383), (1, 4, 1024, 1001)]:
        b, m, k, n = shape
        assert mb.morello_select_path(b, m, k, n) == SK
        A, B, C = w.make(b, m, k, n, seed=1, ab="int4", c="int8")
        got = check_full(A, B, C, integer=True, what="auto %s" % (shape,))
        assert_bit_exact(gpu_run(A, B, C, path=SK, split_k=REG), got, "auto vs forced register kernel")


def test_flat_form_with_more_batches_than_a_grid_dimension():
    b, m, k, n = 66000, 1, 64, 17       # two slabs of batches; every slab starts at another offset
    A, B, C = w.make(b, m, k, n, seed=2, ab="int4", c="int8")
    check_full(A, B, C, integer=True, path=SK, split_k=REG, what="66000 batches")
