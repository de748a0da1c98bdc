"""Seeded random shapes through the selector (and through every forced family that accepts
them) against the CPU oracle: bit-exact on integer inputs.  The shapes mix aligned and
unaligned extents, single rows, few rows, ragged tiles, batches and long k, so that the
selector's every branch (GEMV kernels, operand-swapped kernel with and without k slices,
tile kernels with whole tiles, halves and k slices, row-chunked fallback) is reached."""
import numpy as np
import pytest

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, check_full, gpu_run, to_dev

pytestmark = pytest.mark.gpu


def _shapes(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        b = int(rng.choice([1, 1, 1, 2, 3, 5]))
        m = int(rng.choice([1, 2, 3, 7, 16, 17, 40, 64, 65, 100, 128, 129, 200, 300, 513]))
        kind = rng.integers(0, 4)
        if kind == 0:      # everything a multiple of 8: the TMA-addressable family
            k = 8 * int(rng.integers(1, 400))
            n = 8 * int(rng.integers(1, 300))
        elif kind == 1:    # arbitrary extents: the fallback family
            k = int(rng.integers(1, 1500))
            n = int(rng.integers(1, 1200))
        elif kind == 2:    # long k, few columns: k slices
            k = 64 * int(rng.integers(32, 160))
            n = 8 * int(rng.integers(1, 64))
        else:              # short k, many columns
            k = 8 * int(rng.integers(1, 40))
            n = 8 * int(rng.integers(100, 900))
        if b * m * k * n > 1.2e9:   # keep the oracle within seconds
            m = max(1, int(1.2e9 // (b * k * n)))
        out.append((b, m, k, n))
    return out


@pytest.mark.parametrize("shape", _shapes(20250501, 60))
def test_random_shape_by_selector(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, what="auto %s" % (shape,))
    # Matmul on the same operands: the product alone, whatever C held.
    dA, dB, dC = to_dev(A, B, np.full_like(C, np.nan))
    mb.morello_matmul(b, m, k, n, dA, dB, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, np.zeros_like(C)), "matmul %s" % (shape,))
    # The caller-workspace entry point takes the same route with the advertised size.
    import torch
    need = mb.morello_workspace_bytes(b, m, k, n)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    dA, dB, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_ws(b, m, k, n, dA, dB, dC, ws, need)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), got, "caller workspace %s" % (shape,))


@pytest.mark.parametrize("shape", [s for s in _shapes(7, 40) if s[2] % 8 == 0 and s[3] % 8 == 0])
def test_random_shape_on_every_tensor_form(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="int4", c="int8")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    forms = [1, 2, 16 + 1, 32 + 2, 64 + 1, 64 + 2, 512 * 3 + 1, 512 * 5 + 2]
    if m <= 64:
        forms += [3 + 16, 3 + 32, 3 + 16 + 512 * 4]
    for form in forms:
        got = gpu_run(A, B, C, path=mb.MORELLO_PATH_TCGEN05, split_k=form)
        assert_bit_exact(got, want, "form %d %s" % (form, shape))
    Bt = np.ascontiguousarray(np.swapaxes(B, 1, 2))
    dA, dBt, dC = to_dev(A, Bt, C)
    mb.morello_matmul_accum_colmajor_b(0, b, m, k, n, dA, dBt, dC)
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    assert_bit_exact(dC.cpu().numpy(), want, "column-major B %s" % (shape,))
