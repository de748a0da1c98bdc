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


def test_morello_log_prints_the_route_of_every_call():
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import sys; sys.path.insert(0, %r); import torch\n"
            "from paper_2505_01637_b200 import binding as mb\n"
            "a = torch.zeros(16 * 2048, dtype=torch.int16, device='cuda'); b = torch.zeros(2048 * 1024, dtype=torch.int16, device='cuda')\n"
            "c = torch.zeros(16 * 1024, device='cuda')\n"
            "mb.morello_matmul_accum(1, 16, 2048, 1024, a, b, c); mb.morello_matmul(1, 1, 2048, 1024, a, b, c); torch.cuda.synchronize()\n") % root
    run = subprocess.run([sys.executable, "-c", code], env=dict(os.environ, MORELLO_LOG="1"), capture_output=True,
                         text=True, timeout=300)
    assert run.returncode == 0, run.stderr[-2000:]
    lines = [l for l in run.stderr.splitlines() if l.startswith("morello: ")]
    assert len(lines) == 2
    assert lines[0].startswith("morello: matmul_accum b=1 m=16 k=2048 n=1024 -> tcgen05 swap_kernel")
    assert lines[1].startswith("morello: matmul b=1 m=1 k=2048 n=1024 -> fma ")
