"""GPU parity of the tcgen05 tensor-core path (forced through the C ABI) against
the CPU oracle: single tiles first, then ragged edges, batches, operand-layout pins
and the cross-check against the FP32-FMA path."""
import numpy as np
import pytest

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import assert_bit_exact, bits, check_full, gpu_run

pytestmark = pytest.mark.gpu
TC = mb.MORELLO_PATH_TCGEN05


@pytest.mark.parametrize("shape", [
    (1, 128, 64, 256),      # exactly one tile, one k block
    (1, 128, 16, 256),      # one MMA instruction's worth of k
    (1, 128, 256, 256),     # one tile, the stage ring wraps once
    (1, 128, 640, 256),     # ring wraps several times
    (1, 256, 128, 512),     # 2 x 2 tiles
    (1, 17, 8, 8),          # smallest shape the selector sends here
    (1, 100, 72, 200),      # ragged m, k, n inside one tile
    (1, 129, 200, 264),     # one row / one 8-column group into the next tile
    (2, 300, 520, 776),     # batches with ragged everything
    (3, 64, 64, 64),
    (1, 1024, 128, 2048),   # more tiles than fit one wave of a small grid
])
@pytest.mark.parametrize("form", [1, 2, 16 + 1, 32 + 1, 32 + 2, 64 + 1, 64 + 2,
                                  64 + 2 + 8192 * 1, 32 + 1 + 8192 * 3, 16 + 1 + 8192 * 63])
def test_integer_inputs_bit_exact(shape, form):
    # form % 16: one CTA per tile / a CTA pair per tile; (form // 16) % 16: tile columns / 64 (0 = by
    # shape); form // 8192: rows of tiles per group of the tile order (0 = by shape, 63 = a column
    # of tiles at a time)
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    check_full(A, B, C, integer=True, path=TC, split_k=form, what="tcgen05 form %d %s" % (form, shape))


@pytest.mark.parametrize("shape,form", [
    ((2, 1100, 72, 4504), 64 + 2),    # 180 pair tiles on 74 pairs: the last 32 are cut into halves; ragged n
    ((1, 1280, 72, 4504), 64 + 1),    # 180 one-CTA tiles on 148 SMs: same, halves of 128 columns
    ((1, 4096, 128, 4096), 0),        # the square config's tiling (256 tiles, 34 in the last wave), by shape
    ((1, 2432, 64, 2048), 32 + 1),    # 128-column tiles cut into 64-column halves
])
def test_last_wave_cut_into_column_halves(shape, form):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    cut = check_full(A, B, C, integer=True, path=TC, split_k=form, what="halves %s" % (shape,))
    whole = gpu_run(A, B, C, path=TC, split_k=form + 256)
    assert_bit_exact(whole, cut, "whole tiles vs halves %s" % (shape,))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="normal_rsqrtk", c="normal0.1")
    check_full(A, B, C, integer=False, path=TC, split_k=form, what="halves %s random" % (shape,))


@pytest.mark.parametrize("form", [1, 2])
def test_one_hot_operands_pin_the_operand_layouts(form):
    b, m, k, n = 2, 160, 136, 328
    rng = np.random.default_rng(0)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, i0, p0) in [(0, 0, 0), (0, 37, 70), (1, 159, 135), (1, 128, 64)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Bv[b0, p0, :]
        got = gpu_run(w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Bv), C, path=TC, split_k=form)
        assert_bit_exact(got, want, "one-hot A at %s" % ((b0, i0, p0),))
    for (b0, p0, j0) in [(0, 0, 0), (0, 70, 201), (1, 135, 327), (1, 64, 256)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[b0, p0, j0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        got = gpu_run(w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C, path=TC, split_k=form)
        assert_bit_exact(got, want, "one-hot B at %s" % ((b0, p0, j0),))


def test_identity_operands():
    d = 192
    rng = np.random.default_rng(1)
    X = rng.integers(-100, 101, size=(1, d, d)).astype(np.float32)
    I = np.eye(d, dtype=np.float32)[None]
    C = rng.standard_normal((1, d, d)).astype(np.float32)
    want = (C.astype(np.float64) + X).astype(np.float32)
    assert_bit_exact(gpu_run(w.f32_to_bf16_rne(I), w.f32_to_bf16_rne(X), C, path=TC), want, "A = I")
    assert_bit_exact(gpu_run(w.f32_to_bf16_rne(X), w.f32_to_bf16_rne(I), C, path=TC), want, "B = I")


@pytest.mark.parametrize("shape", [(1, 256, 512, 512), (2, 200, 1000, 328), (1, 128, 4096, 256),
                                   (1, 2048, 2048, 512)])
@pytest.mark.parametrize("form", [1, 2])
def test_random_inputs_within_tolerance(shape, form):
    b, m, k, n = shape
    for ab, c in (("uniform", "normal"), ("normal_rsqrtk", "normal0.1")):
        A, B, C = w.make(b, m, k, n, seed=sum(shape), ab=ab, c=c)
        check_full(A, B, C, integer=False, path=TC, split_k=form,
                   what="tcgen05 form %d %s %s" % (form, shape, ab))


@pytest.mark.parametrize("shape", [(1, 16, 512, 1024), (2, 8, 264, 520), (1, 48, 128, 256)])
def test_both_kernel_families_agree(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=3, ab="int4", c="normal")
    fma = gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY)
    tc = gpu_run(A, B, C, path=TC)
    assert_bit_exact(tc, fma, "tcgen05 vs skinny on integers %s" % (shape,))
    A, B, C = w.make(b, m, k, n, seed=4, ab="uniform", c="normal")
    fma = gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY)
    tc = gpu_run(A, B, C, path=TC)
    T = oracle.abs_dot(b, m, k, n, A, B)
    assert np.all(np.abs(fma.astype(np.float64) - tc) <= 2 * (1e-5 * T + 1e-6))


@pytest.mark.parametrize("form", [1, 2])
def test_repeated_calls_give_identical_bits_and_accumulate(form):
    b, m, k, n = 1, 384, 1024, 768
    A, B, C = w.make(b, m, k, n, seed=5, ab="normal_rsqrtk", c="normal")
    first = gpu_run(A, B, C, path=TC, split_k=form)
    for _ in range(3):
        assert np.array_equal(bits(gpu_run(A, B, C, path=TC, split_k=form)), bits(first))
    A, B, C = w.make(b, m, k, n, seed=6, ab="int4", c="int8")
    twice = oracle.matmul_accum(b, m, k, n, A, B, oracle.matmul_accum(b, m, k, n, A, B, C))
    assert_bit_exact(gpu_run(A, B, C, path=TC, split_k=form, calls=2), twice, "two accumulating calls")


# ------------------------------------------------ the operand-swapped kernel for few rows (form 3)
SWAP = 3


@pytest.mark.parametrize("shape", [
    (1, 1, 64, 128),        # one strip, one k block, one row
    (1, 16, 16, 128),       # one MMA instruction's worth of k
    (1, 3, 640, 256),       # the stage ring wraps
    (2, 16, 200, 264),      # ragged k and n, batches
    (3, 17, 72, 136),       # 17 rows: the 32-row instantiation
    (1, 33, 264, 520),      # 48-row instantiation
    (1, 49, 128, 392),      # 64-row instantiation
    (1, 64, 2048, 1024),
    (2, 60, 136, 264),
    (1, 16, 2048, 16384),   # the decode-style config
])
def test_swap_form_matches_oracle(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    check_full(A, B, C, integer=True, path=TC, split_k=SWAP, what="swap form %s" % (shape,))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="uniform_rsqrtk", c="normal")
    check_full(A, B, C, integer=False, path=TC, split_k=SWAP, what="swap form %s random" % (shape,))


def test_swap_form_one_hot_operands_and_repeatability():
    b, m, k, n = 2, 20, 136, 328
    rng = np.random.default_rng(7)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, i0, p0) in [(0, 0, 0), (0, 19, 70), (1, 7, 135), (1, 16, 64)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Bv[b0, p0, :]
        got = gpu_run(w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Bv), C, path=TC, split_k=SWAP)
        assert_bit_exact(got, want, "swap one-hot A at %s" % ((b0, i0, p0),))
    for (b0, p0, j0) in [(0, 0, 0), (0, 70, 201), (1, 135, 327), (1, 64, 128)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[b0, p0, j0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        got = gpu_run(w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C, path=TC, split_k=SWAP)
        assert_bit_exact(got, want, "swap one-hot B at %s" % ((b0, p0, j0),))
    A, B, C = w.make(1, 16, 1024, 2048, seed=8, ab="normal_rsqrtk", c="normal")
    first = gpu_run(A, B, C, path=TC, split_k=SWAP)
    for _ in range(3):
        assert np.array_equal(bits(gpu_run(A, B, C, path=TC, split_k=SWAP)), bits(first))
    A, B, C = w.make(1, 16, 1024, 2048, seed=9, ab="int4", c="int8")
    twice = oracle.matmul_accum(1, 16, 1024, 2048, A, B, oracle.matmul_accum(1, 16, 1024, 2048, A, B, C))
    assert_bit_exact(gpu_run(A, B, C, path=TC, split_k=SWAP, calls=2), twice, "swap form, two accumulating calls")


@pytest.mark.parametrize("slices", [2, 4, 8])
@pytest.mark.parametrize("shape", [
    (1, 16, 16384, 2048),   # the transposed weight shape: 16 strips, long k
    (2, 3, 1000, 136),      # ragged k blocks, ragged strip, batches
    (1, 64, 4096, 256),     # 64 rows: the accumulator parked in shared memory is 32 KiB
    (1, 33, 520, 392),
])
def test_swap_form_with_k_slices_in_a_cluster(shape, slices):
    b, m, k, n = shape
    knob = SWAP + 16 * slices
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + slices, ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, path=TC, split_k=knob, what="swap, %d slices %s" % (slices, shape))
    assert_bit_exact(gpu_run(A, B, C, path=TC, split_k=SWAP + 16), got, "slices vs one block per strip")
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + slices + 1, ab="uniform_rsqrtk", c="normal")
    first = check_full(A, B, C, integer=False, path=TC, split_k=knob)
    assert np.array_equal(bits(gpu_run(A, B, C, path=TC, split_k=knob)), bits(first))


def test_swap_form_picks_slices_by_shape_and_refuses_odd_counts():
    b, m, k, n = 1, 16, 8192, 1024          # 8 strips: the planner cuts k by itself
    A, B, C = w.make(b, m, k, n, seed=3, ab="int4", c="int8")
    check_full(A, B, C, integer=True, what="auto slices")
    from gpu_util import to_dev
    dA, dB, dC = to_dev(A, B, C)
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(TC, SWAP + 16 * 3, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH


def test_swap_form_refuses_more_than_64_rows():
    b, m, k, n = 1, 65, 64, 128
    A, B, C = w.make(b, m, k, n, seed=1)
    from gpu_util import to_dev
    dA, dB, dC = to_dev(A, B, C)
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(TC, SWAP, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH


# ------------------------------------------------ k slices through the workspace (few tiles, long k)
WS = 512   # knob field: number of k slices whose sums go through the workspace


@pytest.mark.parametrize("slices", [2, 3, 8])
@pytest.mark.parametrize("shape,form", [
    ((1, 128, 2048, 256), 64 + 1),     # one tile of a lone CTA
    ((1, 300, 1000, 520), 64 + 2),     # pair tiles, ragged m, k and n
    ((2, 129, 520, 200), 16 + 1),      # 64-column tiles, batches
    ((1, 256, 4096, 512), 32 + 2),
    ((1, 64, 2048, 384), SWAP + 16),   # operand-swapped, 64 rows
    ((2, 5, 1000, 136), SWAP + 16),    # operand-swapped, ragged, batches
    ((1, 40, 520, 264), SWAP + 16),
])
def test_k_slices_through_the_workspace(shape, form, slices):
    b, m, k, n = shape
    knob = form + WS * slices
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + slices, ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, path=TC, split_k=knob, what="%d slices %s" % (slices, shape))
    assert_bit_exact(gpu_run(A, B, C, path=TC, split_k=form + WS), got, "slices vs whole k")
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + slices + 1, ab="normal_rsqrtk", c="normal")
    first = check_full(A, B, C, integer=False, path=TC, split_k=knob)
    assert np.array_equal(bits(gpu_run(A, B, C, path=TC, split_k=knob)), bits(first))


@pytest.mark.parametrize("shape", [
    (1, 64, 16384, 2048),    # 16 strips of 64 rows: no cluster, slices through the workspace
    (1, 128, 16384, 2048),   # one row of tiles
    (1, 512, 8192, 1024),    # a few pair tiles
    (1, 8, 8192, 8192),      # 64 strips
])
def test_few_tiles_and_a_long_k_by_shape(shape):
    b, m, k, n = shape
    assert mb.morello_workspace_bytes(b, m, k, n) >= 2 * b * m * n * 4
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, what="by shape %s" % (shape,))
    assert np.array_equal(bits(gpu_run(A, B, C)), bits(got))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="normal_rsqrtk", c="normal")
    check_full(A, B, C, integer=False, what="by shape %s random" % (shape,))


def test_k_slices_with_matmul_and_a_caller_workspace():
    from gpu_util import to_dev
    import torch
    b, m, k, n = 1, 128, 4096, 512
    A, B, C = w.make(b, m, k, n, seed=5, ab="int4", c="normal")
    knob = 16 + 1 + WS * 4
    need = mb.morello_workspace_bytes_forced(TC, knob, b, m, k, n)
    assert need == 4 * b * m * n * 4
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    dA, dB, dC = to_dev(A, B, C)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    mb.morello_matmul_accum_forced(TC, knob, b, m, k, n, dA, dB, dC, ws.data_ptr(), need)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), want, "caller workspace")
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(TC, knob, b, m, k, n, dA, dB, dC, ws.data_ptr(), need - 16)
    assert e.value.status == mb.MORELLO_ERR_WORKSPACE
    # Matmul: C = A x B whatever C held.
    dC.fill_(float("nan"))
    mb.morello_matmul_forced(TC, knob, b, m, k, n, dA, dB, dC, 0, 0)
    torch.cuda.synchronize()
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, np.zeros_like(C)), "matmul, slices")


# ------------------------------------------------ operand-swapped kernel, persistent form
@pytest.mark.parametrize("shape", [
    (256, 1, 128, 4096),     # 8,192 items of two k blocks on 296 blocks
    (700, 3, 72, 264),       # ragged k block, ragged strip, items not a multiple of the blocks
    (40, 33, 200, 1000),     # 48-row instantiation: one block per SM
    (66000, 2, 64, 128),     # more batches than a grid dimension
    (3, 16, 4096, 16384),    # long items: 384 items of 64 k blocks
])
def test_swap_form_persistent_blocks_walk_many_items(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape) % 997, ab="int4", c="normal")
    got = check_full(A, B, C, integer=True, path=TC, split_k=SWAP, what="persistent %s" % (shape,))
    assert np.array_equal(bits(gpu_run(A, B, C, path=TC, split_k=SWAP)), bits(got))
    if b * m * k * n < 3e8:
        A, B, C = w.make(b, m, k, n, seed=sum(shape) % 997 + 1, ab="normal_rsqrtk", c="normal")
        check_full(A, B, C, integer=False, path=TC, split_k=SWAP, what="persistent %s random" % (shape,))


def test_swap_form_persistent_with_k_slices_through_the_workspace():
    b, m, k, n = 9, 40, 4096, 520            # 45 strips x 4 slices = 180 items on 148 one-per-SM blocks
    A, B, C = w.make(b, m, k, n, seed=17, ab="int4", c="normal")
    knob = SWAP + 16 + WS * 4
    got = check_full(A, B, C, integer=True, path=TC, split_k=knob, what="persistent, 4 slices")
    assert_bit_exact(gpu_run(A, B, C, path=TC, split_k=SWAP + 16 + WS), got, "slices vs whole k")
