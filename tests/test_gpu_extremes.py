"""GPU parity at the edges of the index arithmetic: more batches than a grid dimension holds,
very wide and very long problems, operands that straddle alignment rules.  Integer inputs,
so every comparison is bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, check_full, to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape", [
    (70000, 1, 8, 8),          # more batches than grid.y holds: slabs of 65,535 (register-streaming kernel)
    (66000, 1, 256, 256),      # same through the TMA-ring GEMV (one tensor map per slab)
    (66000, 2, 64, 128),       # the tensor path takes the batch index from the tile number, no slabs
    (1, 1, 16, 1 << 20),       # a million columns
    (1, 1, 200000, 64),        # a long k on one strip: the planner splits k, the reduce kernel adds the slices
    (1, 3, 40000, 264),
    (1, 2, 8, 100000),         # wide and shallow
    (3, 130, 8, 8),            # one ragged tile per batch
    (1, 5000, 16, 16),         # tall and thin on the tensor path: many m tiles, one n tile
])
def test_extreme_shapes_integer_exact(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape) % 1000, ab="int4", c="int8")
    check_full(A, B, C, integer=True, what="extreme %s" % (shape,))


def test_misaligned_a_or_c_take_the_fma_kernels_with_the_same_result():
    b, m, k, n = 1, 40, 256, 512
    A, B, C = w.make(b, m, k, n, seed=5, ab="int4", c="int8")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    dA, dB, dC = to_dev(A, B, C)
    bigA = torch.zeros(A.size + 8, dtype=torch.int16, device="cuda")
    bigA[1:1 + A.size] = dA.reshape(-1)                    # A two bytes past a 16-byte boundary
    mb.morello_matmul_accum(b, m, k, n, bigA[1:], dB, dC)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), want, "A misaligned for TMA")
    bigC = torch.zeros(C.size + 4, dtype=torch.float32, device="cuda")
    bigC[1:1 + C.size] = torch.from_numpy(C.reshape(-1)).cuda()   # C four bytes past a 16-byte boundary
    mb.morello_matmul_accum(b, m, k, n, dA, dB, bigC[1:])
    torch.cuda.synchronize()
    assert_bit_exact(bigC[1:1 + C.size].cpu().numpy().reshape(b, m, n), want, "C misaligned for TMA")
    assert float(bigC[0]) == 0.0


def test_workspace_query_covers_the_path_a_misaligned_operand_falls_to():
    b, m, k, n = 1, 40, 8192, 64         # aligned: tensor-core tiles, no scratch; A off by 2 bytes: FMA kernel, k in slices
    A, B, C = w.make(b, m, k, n, seed=6, ab="int4", c="int8")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    need = mb.morello_workspace_bytes(b, m, k, n)
    assert need > 0
    dA, dB, dC = to_dev(A, B, C)
    bigA = torch.zeros(A.size + 8, dtype=torch.int16, device="cuda")
    bigA[1:1 + A.size] = dA.reshape(-1)
    ws = torch.empty(need // 4 + 4, device="cuda")
    mb.morello_matmul_accum_ws(b, m, k, n, bigA[1:], dB, dC, ws, need)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), want, "_ws with a misaligned A")
    dC2 = torch.from_numpy(C.copy()).cuda()
    mb.morello_matmul_accum_ws(b, m, k, n, dA, dB, dC2, ws, need)      # aligned: same buffer suffices
    torch.cuda.synchronize()
    assert_bit_exact(dC2.cpu().numpy(), want, "_ws with aligned operands")
