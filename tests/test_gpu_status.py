"""The device status channel: every mbarrier wait in the kernels is bounded; a wait that runs
out records a status word that the host reads as MORELLO_ERR_DEVICE_TIMEOUT, and the context
stays usable.  The library's self-test makes one such wait run out harmlessly (a barrier that
nothing arrives on, a limit of some milliseconds)."""
import time

import numpy as np
import pytest

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, gpu_run

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    assert mb.morello_read_device_status()[0] == mb.MORELLO_OK
    t0 = time.perf_counter()
    mb.morello_selftest_wait_timeout(20)
    assert time.perf_counter() - t0 < 5.0                      # bounded: it gave up by itself
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_ERR_DEVICE_TIMEOUT
    assert detail >> 31 == 1 and (detail >> 16) & 0x7FFF == 0x7E  # the self-test's site code
    assert mb.morello_read_device_status() == (mb.MORELLO_OK, 0)  # reading clears it
    # Ordinary work afterwards: same results, clean status.
    b, m, k, n = 1, 16, 512, 1024
    A, B, C = w.make(b, m, k, n, seed=4, ab="int4", c="normal")
    assert_bit_exact(gpu_run(A, B, C), oracle.matmul_accum(b, m, k, n, A, B, C), "after the self-test")


def test_selftest_rejects_limits_out_of_range():
    for bad in (0, 1001):
        with pytest.raises(mb.MorelloError) as e:
            mb.morello_selftest_wait_timeout(bad)
        assert e.value.status == mb.MORELLO_ERR_INVALID_SHAPE
