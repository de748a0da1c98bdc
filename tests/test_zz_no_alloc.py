"""The allocation-free entry point against the oracle and against the ordinary entry point.

Some users of this library cannot let a call reach cudaMalloc -- their process gave
all device memory to its own pool at start-up, or an allocation's device-wide stall is
not acceptable while serving -- so `morello_matmul_accum_noalloc` keeps the split-k
partial sums in a fixed array inside the library.  This file checks, through the C
ABI, that its result meets the acceptance rule against the CPU oracle (bit-exact on
integer inputs) and has exactly the bits `morello_matmul_accum_forced` gives with the
same split, twice in a row (the array is shared between calls and keeps the previous
call's contents); that a warmed-up call leaves the device's free memory unchanged and is
counted by `morello_launch_count`; and that a problem whose partial sums exceed the array
is refused without touching C.  It is named to be collected after every other test file."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance, to_dev

pytestmark = pytest.mark.gpu


def _both(shape, split_k, dist, seed):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=seed, ab=dist, c="normal")
    dA, dB, dC_ref = to_dev(A, B, C)
    mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, split_k, b, m, k, n, dA, dB, dC_ref)
    _, _, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_noalloc(split_k, b, m, k, n, dA, dB, dC)
    torch.cuda.synchronize()
    got = dC.cpu().numpy()
    want = oracle.matmul_accum(b, m, k, n, A, B, C)         # the oracle decides; the other
    if dist == "int4":                                       # entry point is a second check
        assert_bit_exact(got, want, "no-alloc against the oracle %s" % (shape,))
    else:
        assert_within_tolerance(got, want, oracle.abs_dot(b, m, k, n, A, B),
                                "no-alloc against the oracle %s" % (shape,))
    return got, dC_ref.cpu().numpy()


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    # First call: long k, few columns, split 8.  Second call: another shape and split,
    # so the shared array still holds the first call's partial sums when it starts.
    got, want = _both((1, 4, 8192, 64), 8, "uniform", seed=1)
    assert_bit_exact(got, want, "no-alloc call 1 (split 8)")
    got, want = _both((2, 7, 1000, 72), 3, "int4", seed=2)
    assert_bit_exact(got, want, "no-alloc call 2 (split 3)")
    # the automatic split and more than 16 rows (row chunks share the array in turn)
    got, want = _both((1, 40, 2048, 96), 0, "uniform", seed=3)
    assert_bit_exact(got, want, "no-alloc call 3 (automatic split, 40 rows)")


def test_a_warmed_up_call_allocates_nothing_and_is_counted():
    b, m, k, n, split_k = 1, 4, 8192, 64, 8              # the split needs scratch: 8 x 4 x 64 floats
    A, B, C = w.make(b, m, k, n, seed=6, ab="int4", c="normal")
    dA, dB, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_noalloc(split_k, b, m, k, n, dA, dB, dC)      # loads this kernel variant
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    launches_before = mb.morello_launch_count()
    for _ in range(3):
        mb.morello_matmul_accum_noalloc(split_k, b, m, k, n, dA, dB, dC)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the device's free memory changed across no-alloc calls"
    assert mb.morello_launch_count() - launches_before == 3 * 2        # split kernel + reduce, per call
    want = C
    for _ in range(4):
        want = oracle.matmul_accum(b, m, k, n, A, B, want)
    assert_bit_exact(dC.cpu().numpy(), want, "four accumulating no-alloc calls")


def test_sizes_beyond_the_fixed_array_are_refused():
    limit = mb.morello_noalloc_scratch_limit()
    assert limit == 4 << 20
    b, m, k, n, split_k = 1, 16, 4096, 16384, 8          # 8 * 16 * 16384 * 4 = 8 MiB of partials
    assert split_k * b * m * n * 4 > limit
    A, B, C = w.make(b, m, k, n, seed=4, ab="int4", c="normal")
    dA, dB, dC = to_dev(A, B, C)
    before = dC.clone()
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_noalloc(split_k, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.equal(before, dC)
    # the same problem without a k split needs no scratch at all and is accepted
    mb.morello_matmul_accum_noalloc(1, b, m, k, n, dA, dB, dC)
    ref = before.clone()
    mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, 1, b, m, k, n, dA, dB, ref)
    torch.cuda.synchronize()
    assert torch.equal(ref, dC)
