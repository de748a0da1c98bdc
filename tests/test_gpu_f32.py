"""GPU parity of MatmulAccum on float32 inputs (three-term bf16 split inside the library)
against the CPU oracle for float32 inputs: same acceptance rule as the bf16 operation --
bit-exact when the inputs are bf16-representable integers, otherwise
|gpu - oracle| <= 1e-5 * sum_p |A*B| + 1e-6."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance

pytestmark = pytest.mark.gpu


def _draw(shape, seed, kind):
    b, m, k, n = shape
    rng = np.random.Generator(np.random.Philox(seed))
    if kind == "int":
        A = rng.integers(-4, 5, size=(b, m, k)).astype(np.float32)
        B = rng.integers(-4, 5, size=(b, k, n)).astype(np.float32)
    elif kind == "normal":
        A = (rng.standard_normal((b, m, k)) / np.sqrt(k)).astype(np.float32)
        B = (rng.standard_normal((b, k, n)) / np.sqrt(k)).astype(np.float32)
    else:                       # wide dynamic range: every one of the three terms matters
        A = (rng.standard_normal((b, m, k)) * np.exp2(rng.integers(-6, 7, size=(b, m, k)))).astype(np.float32)
        B = (rng.standard_normal((b, k, n)) * np.exp2(rng.integers(-6, 7, size=(b, k, n)))).astype(np.float32)
    C = rng.standard_normal((b, m, n)).astype(np.float32)
    return A, B, C


def _gpu(shape, A, B, C, calls=1):
    b, m, k, n = shape
    dA, dB, dC = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C.copy()).cuda()
    for _ in range(calls):
        mb.morello_matmul_accum_f32(b, m, k, n, dA, dB, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    return dC.cpu().numpy()


@pytest.mark.parametrize("shape", [
    (1, 4, 4, 16),           # the Figure 1 shape (6k = 24: the tensor path can address it)
    (1, 3, 5, 7),            # nothing a TMA could address: FMA kernels on the split operands
    (2, 40, 63, 36),
    (1, 16, 512, 1024),      # few rows
    (2, 200, 1000, 328),     # ragged tiles, batches
    (1, 256, 512, 512),
    (1, 1, 256, 2048),       # one row
])
def test_f32_inputs_match_oracle(shape):
    b, m, k, n = shape
    A, B, C = _draw(shape, 7 + sum(shape), "int")
    assert_bit_exact(_gpu(shape, A, B, C), oracle.matmul_accum_f32(b, m, k, n, A, B, C), "f32 int %s" % (shape,))
    for kind in ("normal", "wide"):
        A, B, C = _draw(shape, 8 + sum(shape), kind)
        want, T = oracle.matmul_accum_f32(b, m, k, n, A, B, C, want_abs=True)
        assert_within_tolerance(_gpu(shape, A, B, C), want, T, "f32 %s %s" % (kind, shape))


def test_f32_square_2048_sampled_rows():
    """The paper's float32 2048-square matmul at full size; the oracle computes a row sample
    (rows are independent: a row of the result only needs that row of A)."""
    shape = (1, 2048, 2048, 2048)
    b, m, k, n = shape
    A, B, C = _draw(shape, 99, "normal")
    got = _gpu(shape, A, B, C)
    rows = np.r_[0:16, 1016:1032, 2032:2048, np.random.default_rng(0).integers(0, m, 48)]
    As, Cs = np.ascontiguousarray(A[:, rows, :]), np.ascontiguousarray(C[:, rows, :])
    want, T = oracle.matmul_accum_f32(b, len(rows), k, n, As, B, Cs, want_abs=True)
    ratio = assert_within_tolerance(got[:, rows, :], want, T, "f32 2048-square")
    assert ratio < 0.5          # the split leaves the f32 accumulation error, far inside the bound
    assert np.isfinite(got).all()


def test_f32_calls_accumulate_and_repeat_bit_for_bit():
    shape = (1, 192, 256, 384)
    b, m, k, n = shape
    A, B, C = _draw(shape, 5, "int")
    twice = oracle.matmul_accum_f32(b, m, k, n, A, B, oracle.matmul_accum_f32(b, m, k, n, A, B, C))
    assert_bit_exact(_gpu(shape, A, B, C, calls=2), twice, "two accumulating f32 calls")
    A, B, C = _draw(shape, 6, "normal")
    first = _gpu(shape, A, B, C)
    for _ in range(2):
        assert np.array_equal(_gpu(shape, A, B, C).view(np.uint32), first.view(np.uint32))


def test_f32_empty_and_bad_arguments():
    dA = torch.zeros(64, device="cuda")
    dC = torch.full((2, 8), 3.0, device="cuda")
    mb.morello_matmul_accum_f32(1, 2, 0, 8, dA, dA, dC)          # empty sum: C untouched
    torch.cuda.synchronize()
    assert torch.all(dC == 3.0)
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_f32(1, -2, 4, 8, dA, dA, dC)
    assert e.value.status == mb.MORELLO_ERR_INVALID_SHAPE


@pytest.mark.parametrize("shape", [
    (1, 256, 512, 512),      # tile kernel
    (2, 16, 1024, 1024),     # operand-swapped kernel
    (1, 8, 4096, 256),       # ... with k slices inside a cluster
    (1, 300, 4096, 264),     # tile kernel with k slices through the workspace
    (1, 64, 64, 128),        # one k block per term
    (40, 16, 128, 1024),     # 320 (batch, strip) items: the operand-swapped kernel's persistent form
])
def test_f32_three_stored_terms_equal_the_six_term_problem(shape):
    """With k % 64 == 0 the library stores the three bf16 terms of A and B once and lets the
    tensor kernels visit them in the six-product order.  The same six products laid out in
    full on the host and run as a plain bf16 problem of 6k must give the same bits."""
    b, m, k, n = shape
    A, B, C = _draw(shape, 21 + sum(shape), "wide")

    def terms(x):
        h1 = w.f32_to_bf16_rne(x)
        r1 = x - w.bf16_to_f32(h1)
        h2 = w.f32_to_bf16_rne(r1)
        r2 = r1 - w.bf16_to_f32(h2)
        return h1, h2, w.f32_to_bf16_rne(r2)

    a1, a2, a3 = terms(A)
    b1, b2, b3 = terms(B)
    A6 = np.ascontiguousarray(np.concatenate([a3, a1, a2, a2, a1, a1], axis=2))
    B6 = np.ascontiguousarray(np.concatenate([b1, b3, b2, b1, b2, b1], axis=1))
    from gpu_util import gpu_run
    plain = gpu_run(A6, B6, C)
    assert np.array_equal(_gpu(shape, A, B, C).view(np.uint32), plain.view(np.uint32))


@pytest.mark.parametrize("shape", [(1, 256, 512, 512), (2, 40, 63, 36), (1, 16, 1024, 1024)])
def test_f32_matmul_never_reads_c(shape):
    b, m, k, n = shape
    A, B, C = _draw(shape, 41 + sum(shape), "int")
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    dC = torch.full((b, m, n), float("nan"), device="cuda")
    mb.morello_matmul_f32(b, m, k, n, dA, dB, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum_f32(b, m, k, n, A, B, np.zeros_like(C)), "f32 matmul %s" % (shape,))
    dC.fill_(5.0)
    mb.morello_matmul_f32(b, m, 0, n, dA, dB, dC)          # an empty sum: C = 0
    torch.cuda.synchronize()
    assert float(dC.abs().max()) == 0.0
