"""GPU parity of the non-accumulating Matmul entry point (C = A x B, C's prior contents
ignored) against the CPU oracle applied to a zeroed output, on every kernel family."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance, to_dev

pytestmark = pytest.mark.gpu
SK, TC = mb.MORELLO_PATH_SKINNY, mb.MORELLO_PATH_TCGEN05

CASES = [
    # (path, knob, shape)
    (SK, 1024, (2, 5, 300, 1000)),         # register-streaming kernel, one k slice
    (SK, 1024 + 4, (1, 3, 1024, 72)),      # ... with k slices and the reduce kernel
    (SK, 1024, (1, 40, 64, 36)),           # ... rows in chunks of 16, nothing TMA could address
    (SK, 2048, (1, 1, 2048, 4096)),        # TMA-ring GEMV
    (SK, 2048 + 3, (2, 2, 1000, 264)),     # ... with k slices
    (TC, 3, (2, 16, 200, 264)),            # operand-swapped kernel
    (TC, 3, (1, 50, 136, 264)),            # ... the 200 KiB ring
    (TC, 3 + 16 * 4, (1, 16, 2048, 264)),  # ... four k slices in a cluster
    (TC, 1, (1, 100, 72, 200)),            # one-CTA tiles, ragged
    (TC, 2, (2, 300, 520, 776)),           # CTA-pair tiles, ragged
    (TC, 64 + 2, (2, 1100, 72, 4504)),     # last wave cut into halves
    (mb.MORELLO_PATH_AUTO, 0, (1, 1, 2048, 16384)),
    (mb.MORELLO_PATH_AUTO, 0, (1, 16, 2048, 16384)),
]


@pytest.mark.parametrize("path,knob,shape", CASES)
def test_matmul_overwrites_c(path, knob, shape):
    b, m, k, n = shape
    for dist, integer in (("int4", True), ("uniform", False)):
        A, B, _ = w.make(b, m, k, n, seed=sum(shape) + knob, ab=dist, c="zeros")
        zeros = np.zeros((b, m, n), np.float32)
        want = oracle.matmul_accum(b, m, k, n, A, B, zeros)
        dA, dB, _ = to_dev(A, B, zeros)
        # whatever C held must not matter: poison it (NaN would survive any addition)
        dC = torch.full((b, m, n), float("nan"), device="cuda")
        mb.morello_matmul_forced(path, knob, b, m, k, n, dA, dB, dC)
        st, detail = mb.morello_read_device_status()
        assert st == mb.MORELLO_OK, hex(detail)
        got = dC.cpu().numpy()
        if integer:
            assert_bit_exact(got, want, "matmul %s knob %d" % (shape, knob))
        else:
            assert_within_tolerance(got, want, oracle.abs_dot(b, m, k, n, A, B), "matmul %s" % (shape,))


def test_matmul_with_empty_k_zeroes_c_and_empty_outputs_do_nothing():
    dA, dB, _ = to_dev(*w.make(1, 2, 4, 8, seed=1))
    dC = torch.full((1, 2, 8), 7.0, device="cuda")
    launches = mb.morello_launch_count()
    mb.morello_matmul(1, 2, 0, 8, dA, dB, dC)
    torch.cuda.synchronize()
    assert torch.all(dC == 0) and mb.morello_launch_count() == launches
    dC.fill_(7.0)
    for shape in [(0, 2, 4, 8), (1, 0, 4, 8), (1, 2, 4, 0)]:
        mb.morello_matmul(*shape, dA, dB, dC)
    torch.cuda.synchronize()
    assert torch.all(dC == 7.0)


def test_matmul_then_accumulate_equals_twice_the_product():
    b, m, k, n = 1, 192, 256, 384
    A, B, _ = w.make(b, m, k, n, seed=5, ab="int4", c="zeros")
    zeros = np.zeros((b, m, n), np.float32)
    once = oracle.matmul_accum(b, m, k, n, A, B, zeros)
    twice = oracle.matmul_accum(b, m, k, n, A, B, once)
    dA, dB, _ = to_dev(A, B, zeros)
    dC = torch.full((b, m, n), float("nan"), device="cuda")
    mb.morello_matmul(b, m, k, n, dA, dB, dC)
    mb.morello_matmul_accum(b, m, k, n, dA, dB, dC)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), twice, "matmul followed by matmul_accum")
