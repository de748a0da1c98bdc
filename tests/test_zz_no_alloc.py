"""The allocation-free entry point gives the same bits as the ordinary one.

Some users of this library cannot let a call reach cudaMalloc -- their process gave
all device memory to its own pool at start-up, or an allocation's device-wide stall is
not acceptable while serving -- so `morello_matmul_accum_noalloc` keeps the split-k
partial sums in a fixed array inside the library.  This file checks, through the C
ABI, that it computes exactly what `morello_matmul_accum_forced` computes with the
same split, twice in a row (the array is shared between calls and keeps the previous
call's contents), and that a problem whose partial sums exceed the array is refused
without touching C.  It is named to be collected after every other test file."""
import numpy as np
import pytest
import torch

from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, to_dev

pytestmark = pytest.mark.gpu


def _both(shape, split_k, dist, seed):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=seed, ab=dist, c="normal")
    dA, dB, dC_ref = to_dev(A, B, C)
    mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, split_k, b, m, k, n, dA, dB, dC_ref)
    _, _, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_noalloc(split_k, b, m, k, n, dA, dB, dC)
    torch.cuda.synchronize()
    return dC.cpu().numpy(), dC_ref.cpu().numpy()


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
