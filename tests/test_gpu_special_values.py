"""IEEE special values through every kernel family, against the CPU oracle: bf16 subnormal
inputs, products that are float32 subnormals, infinities of both signs, NaN operands,
Inf x 0 and Inf - Inf.  The definition (Section 2.2's Matmul, accumulating form) is a sum of
products, so IEEE 754 fixes each of these results; the oracle is pinned to them by hand in
the CPU tests, and here every route must produce NaN exactly where the oracle does and the
oracle's bits (infinities and subnormals included) everywhere else -- no flush to zero, no
NaN leaking into another row or column of a tile.  The one documented exception: where the
tensor-core kernels add into a C that the TMA engine cannot address, the final addition is a
reduction in L2 that takes subnormal operands and results for zero; that route is held to the
oracle's result with its subnormals replaced by zeros of the same sign."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import bits, to_dev

pytestmark = pytest.mark.gpu


def assert_same_specials(got, want, what):
    nan_g, nan_w = np.isnan(got), np.isnan(want)
    if not np.array_equal(nan_g, nan_w):
        bad = np.argwhere(nan_g != nan_w)
        raise AssertionError("%s: NaN pattern differs at %d elements; first %s: got %r want %r" % (
            what, len(bad), tuple(bad[0]), got[tuple(bad[0])], want[tuple(bad[0])]))
    rest = ~nan_w
    gb, wb = bits(got)[rest], bits(want)[rest]
    if not np.array_equal(gb, wb):
        bad = np.flatnonzero(gb != wb)
        raise AssertionError("%s: %d elements differ outside the NaNs; first got 0x%08x want 0x%08x" % (
            what, len(bad), gb[bad[0]], wb[bad[0]]))


def subnormals_flushed(x):
    out = x.copy()
    tiny = (np.abs(out) < np.float32(2.0 ** -126)) & (out != 0)
    out[tiny] = np.copysign(np.float32(0), out[tiny])
    return out


def device_ok():
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)


SHAPES = [
    (1, 256, 512),        # streaming GEMV, one k slice
    (1, 16384, 2048),     # streaming GEMV, k slices in a cluster
    (1, 2048, 16384),     # the headline shape
    (1, 255, 515),        # one row, extents the TMA engine cannot address: register streaming
    (3, 255, 515),        # few rows, the same
    (2, 256, 512),        # operand-swapped tensor kernel, 16 rows per MMA
    (16, 2048, 1024),     # the same with k slices
    (40, 256, 512),       # 48 rows per MMA
    (64, 2048, 2048),     # 64 rows, k slices through the workspace
    (128, 256, 512),      # tile kernel, one CTA per tile
    (200, 136, 776),      # ragged tiles
    (512, 8192, 264),     # tile kernel, k slices through the workspace
    (1536, 128, 2816),    # CTA pairs
    (40, 255, 515),       # more than 16 rows, not TMA-addressable: padded copies or row chunks
    (300, 1000, 1003),    # padded copies, C written from registers
]


@pytest.mark.parametrize("shape", SHAPES)
def test_every_route_handles_special_values_like_the_oracle(shape):
    m, k, n = shape
    firsts = range(6) if m == 1 else (0, 2)
    for first in firsts:
        A, B, C, kinds = w.make_special(m, k, n, seed=31 * m + k + n, first=first)
        want = oracle.matmul_accum(1, m, k, n, A, B, C)
        assert np.isnan(want).any() and (m < 7 or np.isinf(want).any())
        route = mb.morello_describe_route(1, m, k, n)
        dA, dB, dC = to_dev(A, B, C)
        mb.morello_matmul_accum(1, m, k, n, dA, dB, dC)
        in_l2 = "C written from registers" in route and "gemm_kernel" in route
        assert in_l2 or shape != (300, 1000, 1003), route
        assert_same_specials(dC.cpu().numpy(), subnormals_flushed(want) if in_l2 else want,
                             "%s first %d (%s)" % (shape, first, route))
        for path in (mb.MORELLO_PATH_SKINNY, mb.MORELLO_PATH_TCGEN05):
            if path == mb.MORELLO_PATH_TCGEN05 and (k % 8 or n % 8):
                continue
            dA, dB, dC = to_dev(A, B, C)
            mb.morello_matmul_accum_forced(path, 0, 1, m, k, n, dA, dB, dC)
            assert_same_specials(dC.cpu().numpy(), want, "%s first %d forced path %d" % (shape, first, path))
        device_ok()


@pytest.mark.parametrize("shape", [(1, 2048, 4096), (16, 520, 776), (300, 1000, 328), (1536, 128, 2816), (5, 33, 50)])
def test_other_entry_points_handle_special_values_like_the_oracle(shape):
    m, k, n = shape
    A, B, C, kinds = w.make_special(m, k, n, seed=7 * m + k + n, first=1)
    want = oracle.matmul_accum(1, m, k, n, A, B, C)
    # Matmul: C is overwritten, whatever it held
    dA, dB, dC = to_dev(A, B, np.full_like(C, 123.0))
    mb.morello_matmul(1, m, k, n, dA, dB, dC)
    assert_same_specials(dC.cpu().numpy(), oracle.matmul_accum(1, m, k, n, A, B, np.zeros_like(C)), "matmul %s" % (shape,))
    # column-major B
    Bt = np.ascontiguousarray(np.swapaxes(B, 1, 2))
    dA, dBt, dC = to_dev(A, Bt, C)
    mb.morello_matmul_accum_colmajor_b(0, 1, m, k, n, dA, dBt, dC)
    assert_same_specials(dC.cpu().numpy(), want, "column-major B %s" % (shape,))
    # B packed in strips of 64 columns (padding of the last strip: NaN patterns that must not be read)
    Bp = w.pack_b(B, 64, fill=w.BF16_QUIET_NAN)
    dA, dBp, dC = to_dev(A, Bp, C)
    mb.morello_matmul_accum_packed_b(64, 1, m, k, n, dA, dBp, dC)
    assert_same_specials(dC.cpu().numpy(), want, "packed B %s" % (shape,))
    # caller's workspace
    need = mb.morello_workspace_bytes(1, m, k, n)
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    dA, dB, dC = to_dev(A, B, C)
    mb.morello_matmul_accum_ws(1, m, k, n, dA, dB, dC, ws, need)
    assert_same_specials(dC.cpu().numpy(), want, "_ws %s" % (shape,))
    device_ok()


def test_float32_entry_keeps_subnormals_and_answers_infinities_with_nan():
    """The three-term bf16 split of the float32 entry point is exact on bf16-representable
    inputs, subnormal ones included; an infinite input splits into Inf, NaN, NaN (Inf - Inf), so
    every sum it reaches is NaN where the definition gives an infinity."""
    m, k, n = 300, 1024, 512
    A, B, C, kinds = w.make_special(m, k, n, seed=11, first=0)
    Af, Bf = w.bf16_to_f32(A), w.bf16_to_f32(B)
    want = oracle.matmul_accum_f32(1, m, k, n, Af, Bf, C)
    dA, dB = torch.from_numpy(Af).cuda(), torch.from_numpy(Bf).cuda()
    dC = torch.from_numpy(C.copy()).cuda()
    mb.morello_matmul_accum_f32(1, m, k, n, dA, dB, dC)
    got = dC.cpu().numpy()
    device_ok()
    finite = np.isfinite(want)
    assert np.array_equal(bits(got)[finite], bits(want)[finite])       # subnormal rows and ordinary rows
    assert finite[0, [kinds.index("subnormal_input"), kinds.index("subnormal_product")], :6].all()
    assert np.isnan(got[~finite]).all()                                # NaN and +-Inf alike
    assert np.isinf(want).any()
