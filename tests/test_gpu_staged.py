"""Extents the TMA engine cannot address (k % 8 != 0 or n % 8 != 0) with more than a few rows:
the selector copies the operands into zero-padded buffers and runs the tensor-core kernels on
those.  Parity with the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, assert_within_tolerance, bits, check_full, gpu_run, to_dev

pytestmark = pytest.mark.gpu

SHAPES = [
    (1, 512, 1000, 1001),    # both extents odd
    (1, 300, 1001, 1000),    # only k: C is added to directly
    (1, 300, 1000, 1001),    # only n: A is used as it is
    (2, 130, 517, 1234),     # batches; n % 4 == 2
    (3, 20, 2000, 999),      # few rows: the operand-swapped kernel behind the copies
    (1, 100, 9000, 260 + 3), # long k, few columns: k slices behind the copies
    (1, 1025, 70, 2051),
    (1, 17, 100, 100),       # small: two chunks of rows on the FMA kernels would cost more
    (2, 260, 72, 1003),      # A is used as it is, C written from registers by CTA pairs, two batches
    (1, 200, 8200, 303),     # tile kernel with k slices: the reduce launch narrows 304 columns to 303
]


@pytest.mark.parametrize("shape", SHAPES)
def test_padded_copies_match_the_oracle(shape):
    b, m, k, n = shape
    assert mb.morello_select_path(b, m, k, n) == mb.MORELLO_PATH_TCGEN05
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, what="padded copies %s" % (shape,))
    # The FMA kernels on the same operands: same bits on integer inputs.
    assert_bit_exact(gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY), got, "FMA path vs padded copies")
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="normal_rsqrtk", c="normal")
    first = check_full(A, B, C, integer=False, what="padded copies %s random" % (shape,))
    assert np.array_equal(bits(gpu_run(A, B, C)), bits(first))


def test_padded_copies_matmul_and_caller_workspace():
    b, m, k, n = 2, 200, 333, 777
    A, B, C = w.make(b, m, k, n, seed=11, ab="int4", c="normal")
    dA, dB, dC = to_dev(A, B, np.full_like(C, np.nan))
    mb.morello_matmul(b, m, k, n, dA, dB, dC)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, np.zeros_like(C)), "matmul")
    need = mb.morello_workspace_bytes(b, m, k, n)
    copies = 2 * b * m * 336 + 2 * b * 336 * 784           # A' and B'; C is written in place
    assert copies <= need < copies + 4 * b * m * 784
    ws = torch.empty(need + 16, dtype=torch.uint8, device="cuda")
    dA, dB, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_ws(b, m, k, n, dA, dB, dC, ws.data_ptr() + 16, need)   # 16-byte aligned only
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, C), "caller workspace")
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_ws(b, m, k, n, dA, dB, dC, ws.data_ptr(), 1024)
    assert e.value.status == mb.MORELLO_ERR_WORKSPACE
    # Forcing the tensor path means the direct kernels: they refuse the shape.
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(mb.MORELLO_PATH_TCGEN05, 0, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH


def test_padded_copies_with_operands_at_odd_addresses():
    # k % 8 != 0, n % 8 == 0: C would be used directly, but here it starts 4 bytes off a
    # 16-byte boundary (and A, B 2 bytes off): every operand goes through a copy.
    b, m, k, n = 1, 64, 1003, 512
    A, B, C = w.make(b, m, k, n, seed=5, ab="int4", c="normal")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    bufA = torch.zeros(A.size + 8, dtype=torch.int16, device="cuda")
    bufB = torch.zeros(B.size + 8, dtype=torch.int16, device="cuda")
    bufC = torch.zeros(C.size + 8, dtype=torch.float32, device="cuda")
    dA = bufA[1:1 + A.size]; dA.copy_(torch.from_numpy(A.view(np.int16).reshape(-1)))
    dB = bufB[1:1 + B.size]; dB.copy_(torch.from_numpy(B.view(np.int16).reshape(-1)))
    dC = bufC[1:1 + C.size]; dC.copy_(torch.from_numpy(C.reshape(-1)))
    assert dA.data_ptr() % 16 == 2 and dC.data_ptr() % 16 == 4
    mb.morello_matmul_accum(b, m, k, n, dA.data_ptr(), dB.data_ptr(), dC.data_ptr())
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy().reshape(C.shape), want, "odd addresses")
    assert float(bufC[0]) == 0.0 and float(bufC[1 + C.size]) == 0.0      # nothing written outside C


def test_small_or_few_row_shapes_keep_the_fma_kernels():
    for shape in [(1, 2, 2048, 1001), (1, 16, 100, 100), (1, 1, 2047, 16383)]:
        assert mb.morello_select_path(*shape) == mb.MORELLO_PATH_SKINNY
        A, B, C = w.make(*shape, seed=3, ab="int4", c="int8")
        check_full(A, B, C, integer=True, what="%s" % (shape,))


@pytest.mark.filterwarnings("ignore:The CUDA Graph is empty")
def test_growing_a_library_buffer_inside_a_stream_capture_is_refused_cleanly():
    # The float32 entry point keeps its split operands in a library-owned buffer that grows by
    # cudaFree + cudaMalloc, which a capturing stream does not allow: the call is refused with
    # MORELLO_ERR_WORKSPACE before anything touches the device, the capture stays valid, and once an
    # ordinary call has sized the buffer the same call captures and replays correctly.
    b, m, k, n = 1, 192, 3136, 3072            # 12 bytes per element of A and B: a buffer no other test needs
    rng = np.random.default_rng(5)
    A = rng.integers(-4, 5, size=(b, m, k)).astype(np.float32)
    B = rng.integers(-4, 5, size=(b, k, n)).astype(np.float32)
    C = rng.standard_normal((b, m, n)).astype(np.float32)
    dA, dB, dC = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), torch.from_numpy(C.copy()).cuda()
    call = mb.lib().morello_matmul_accum_f32
    mb.morello_device_limits()                 # the library's per-device set-up, outside any capture
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            rc = call(b, m, k, n, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), side.cuda_stream)
    assert rc == mb.MORELLO_ERR_WORKSPACE, rc
    g.replay()                                   # an empty graph: the capture survived the refusal
    torch.cuda.synchronize()
    assert torch.equal(dC, torch.from_numpy(C).cuda())
    mb.morello_matmul_accum_f32(b, m, k, n, dA, dB, dC)          # sizes the buffer
    torch.cuda.synchronize()
    want = oracle.matmul_accum_f32(b, m, k, n, A, B, C)
    assert_bit_exact(dC.cpu().numpy(), want, "float32, integer-valued inputs")
    g2 = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g2, stream=side):
            rc = call(b, m, k, n, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), side.cuda_stream)
    assert rc == mb.MORELLO_OK
    g2.replay()
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum_f32(b, m, k, n, A, B, want), "captured call replayed")
