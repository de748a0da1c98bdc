"""GPU parity: the CUDA path through the C ABI against the CPU oracle,
element by element, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_01637_b200 import binding as mb
from paper_2505_01637_b200 import workloads as w

from gpu_util import (assert_bit_exact, assert_within_tolerance, bits, check_full, check_rows,
                      gpu_run, to_dev)

pytestmark = pytest.mark.gpu


# ---------------------------------------------------- T1: tiny and odd shapes
@pytest.mark.parametrize("m", list(range(1, 18)) + [33])
def test_every_row_count_integer_exact(m):
    for (b, k, n) in [(1, 64, 128), (2, 65, 72), (3, 7, 24)]:
        A, B, C = w.make(b, m, k, n, seed=100 + m, ab="int4", c="normal")
        check_full(A, B, C, integer=True, what="m=%d b=%d k=%d n=%d" % (m, b, k, n))


@pytest.mark.parametrize("k", [1, 2, 3, 4, 7, 8, 9, 63, 64, 65, 127, 129, 1000])
@pytest.mark.parametrize("n", [1, 2, 3, 4, 6, 8, 12, 20, 100, 257])
def test_odd_k_and_n(k, n):
    for m in (1, 3, 16):
        A, B, C = w.make(2, m, k, n, seed=7 * k + n, ab="int4", c="int8")
        check_full(A, B, C, integer=True, what="m=%d k=%d n=%d" % (m, k, n))


@pytest.mark.parametrize("shape", [(1, 1, 512, 2048), (2, 5, 300, 1000), (1, 16, 1024, 4096),
                                   (3, 9, 2050, 264), (1, 40, 256, 520), (1, 2, 4096, 96)])
def test_random_inputs_within_tolerance(shape):
    b, m, k, n = shape
    for ab, c in (("uniform", "normal"), ("normal_rsqrtk", "normal0.1")):
        A, B, C = w.make(b, m, k, n, seed=sum(shape), ab=ab, c=c)
        check_full(A, B, C, integer=False, what=str(shape))


def test_one_hot_operands_pin_layout():
    b, m, k, n = 3, 5, 24, 40
    rng = np.random.default_rng(0)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, i0, p0) in [(0, 0, 0), (1, 2, 13), (2, 4, 23)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Bv[b0, p0, :]
        got = gpu_run(w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Bv), C)
        assert_bit_exact(got, want, "one-hot A at %s" % ((b0, i0, p0),))
    for (b0, p0, j0) in [(0, 0, 0), (1, 13, 22), (2, 23, 39)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[b0, p0, j0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        got = gpu_run(w.f32_to_bf16_rne(Av), w.f32_to_bf16_rne(B1), C)
        assert_bit_exact(got, want, "one-hot B at %s" % ((b0, p0, j0),))


# --------------------------------------------------- T2: the five configurations
@pytest.mark.parametrize("index", [0, 1, 2])
@pytest.mark.parametrize("variant", ["random", "integer", "integer_intc"])
def test_configs_1_to_3_full(index, variant):
    A, B, C = w.make_config(index, variant)
    check_full(A, B, C, integer=(variant != "random"),
               what="%s/%s" % (w.CONFIGS[index].name, variant))


@pytest.mark.parametrize("variant", ["random", "integer"])
def test_config_4_whole_output(variant):
    A, B, C = w.make_config(3, variant)
    check_full(A, B, C, integer=(variant != "random"), what="%s/%s" % (w.CONFIGS[3].name, variant))


@pytest.mark.parametrize("index", [3, 4])
@pytest.mark.parametrize("variant", ["random", "integer"])
def test_configs_4_and_5_sampled_rows(index, variant):
    cfg = w.CONFIGS[index]
    A, B, C = w.make_config(index, variant)
    got = gpu_run(A, B, C)
    rows = w.sample_rows(cfg.b, cfg.m, seed=index)
    check_rows(A, B, C, rows, integer=(variant != "random"), got=got,
               what="%s/%s" % (cfg.name, variant))
    if cfg.c == "zeros":     # untouched-input property that holds at any size
        assert np.isfinite(got).all()


# -------------------------------------------- T3: split-k and workspace variants
@pytest.mark.parametrize("split_k", [1, 2, 3, 8, 32])
def test_forced_split_k_matches_oracle(split_k):
    for (b, m, k, n) in [(1, 1, 2048, 256), (2, 7, 1000, 72), (1, 16, 4096, 64)]:
        A, B, C = w.make(b, m, k, n, seed=split_k, ab="int4", c="normal")
        check_full(A, B, C, integer=True, path=mb.MORELLO_PATH_SKINNY, split_k=split_k,
                   what="split %d %s" % (split_k, (b, m, k, n)))
        A, B, C = w.make(b, m, k, n, seed=split_k, ab="uniform", c="normal")
        check_full(A, B, C, integer=False, path=mb.MORELLO_PATH_SKINNY, split_k=split_k)


def test_caller_workspace_and_its_size_check():
    b, m, k, n = 1, 4, 8192, 64          # few columns, long k: the register-streaming kernel splits k
    REG = 1024                           # that kernel, split by shape
    A, B, C = w.make(b, m, k, n, seed=5, ab="int4", c="normal")
    need = mb.morello_workspace_bytes_forced(mb.MORELLO_PATH_SKINNY, REG, b, m, k, n)
    assert need > 0 and mb.morello_workspace_bytes(b, m, k, n) >= need
    dA, dB, dC = to_dev(A, B, C)
    ws = torch.full((need // 4 + 64,), float("nan"), device="cuda")   # poisoned scratch
    mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, REG, b, m, k, n, dA, dB, dC, ws, need)
    assert_bit_exact(dC.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, C), "caller's scratch")
    assert torch.isnan(ws[need // 4:]).all()                          # nothing past the stated size
    before = dC.clone()
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, REG, b, m, k, n, dA, dB, dC, ws, need - 4)
    assert e.value.status == mb.MORELLO_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.equal(before, dC)
    # the selector's own choice for this shape needs no scratch at all; the _ws call takes any
    dC2 = torch.from_numpy(C.copy()).cuda()
    mb.morello_matmul_accum_ws(b, m, k, n, dA, dB, dC2, ws, need)
    torch.cuda.synchronize()
    assert_bit_exact(dC2.cpu().numpy(), oracle.matmul_accum(b, m, k, n, A, B, C), "ws variant")


# ------------------------------------- T3b: the TMA-ring GEMV kernel, forced (knob 2048 + split)
STREAM = 2 * 1024


@pytest.mark.parametrize("shape", [
    (1, 1, 64, 64),          # one box
    (1, 1, 2048, 16384),     # the headline shape
    (1, 1, 100, 72),         # ragged k (scalar staging of A) and a partial last strip
    (2, 3, 1000, 200),       # batches, m = 3 in the 4-row kernel, k % 8 == 0 but ragged boxes
    (3, 2, 321, 136),
    (1, 4, 5000, 328),       # k longer than one block's slice: the planner splits k
    (1, 4, 2048, 4096),
    (2, 1, 8192, 64),        # few strips, long k
])
def test_stream_kernel_matches_oracle(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=sum(shape), ab="int4", c="normal")
    check_full(A, B, C, integer=True, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM, what="stream %s" % (shape,))
    A, B, C = w.make(b, m, k, n, seed=sum(shape) + 1, ab="uniform", c="normal")
    check_full(A, B, C, integer=False, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM, what="stream %s" % (shape,))


@pytest.mark.parametrize("split_k", [1, 2, 3, 7, 8, 32])
@pytest.mark.parametrize("kernel", [STREAM, STREAM + 1024])     # slices added in a cluster / from scratch
def test_stream_kernel_forced_splits(split_k, kernel):
    for (b, m, k, n) in [(1, 1, 2048, 256), (2, 3, 1000, 72), (1, 4, 4096, 64)]:
        A, B, C = w.make(b, m, k, n, seed=split_k, ab="int4", c="normal")
        got = check_full(A, B, C, integer=True, path=mb.MORELLO_PATH_SKINNY, split_k=kernel + split_k,
                         what="stream split %d %s" % (split_k, (b, m, k, n)))
        A, B, C = w.make(b, m, k, n, seed=split_k + 1, ab="uniform", c="normal")
        check_full(A, B, C, integer=False, path=mb.MORELLO_PATH_SKINNY, split_k=kernel + split_k)


def test_stream_kernel_cluster_reduce_needs_no_scratch_and_repeats():
    b, m, k, n = 1, 1, 16384, 2048          # few strips, long k: eight slices per strip, one cluster each
    assert mb.morello_workspace_bytes_forced(mb.MORELLO_PATH_SKINNY, STREAM, b, m, k, n) == 0
    assert mb.morello_workspace_bytes_forced(mb.MORELLO_PATH_SKINNY, STREAM + 1024, b, m, k, n) > 0
    A, B, C = w.make(b, m, k, n, seed=77, ab="int4", c="normal")
    check_full(A, B, C, integer=True, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM, what="cluster reduce")
    A, B, C = w.make(b, m, k, n, seed=78, ab="uniform", c="normal")
    first = gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM, calls=3)
    again = gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM, calls=3)
    assert np.array_equal(bits(first), bits(again))


def test_stream_kernel_one_hot_and_repeatability():
    b, m, k, n = 2, 2, 192, 136
    rng = np.random.default_rng(3)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    for (b0, i0, p0) in [(0, 0, 0), (1, 1, 191), (0, 1, 64)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Bv[b0, p0, :]
        got = gpu_run(w.f32_to_bf16_rne(A1), w.f32_to_bf16_rne(Bv), C, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM)
        assert_bit_exact(got, want, "stream one-hot A at %s" % ((b0, i0, p0),))
    A, B, C = w.make(1, 1, 2048, 16384, seed=21, ab="uniform", c="normal")
    first = gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM)
    for _ in range(3):
        assert np.array_equal(bits(gpu_run(A, B, C, path=mb.MORELLO_PATH_SKINNY, split_k=STREAM)), bits(first))


def test_stream_kernel_refuses_what_it_cannot_address():
    b, m, k, n = 1, 2, 64, 36             # n not a multiple of 8
    dA, dB, dC = to_dev(*w.make(b, m, k, n, seed=13))
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, STREAM, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH
    dA, dB, dC = to_dev(*w.make(1, 5, 64, 64, seed=13))      # more than 4 rows
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(mb.MORELLO_PATH_SKINNY, STREAM, 1, 5, 64, 64, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH


# ------------------------------------------------------------- T4: determinism
@pytest.mark.parametrize("shape", [(1, 1, 2048, 16384), (1, 16, 2048, 1024), (1, 3, 8192, 64)])
def test_repeated_calls_give_identical_bits(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=9, ab="uniform", c="normal")
    first = gpu_run(A, B, C)
    for _ in range(3):
        assert np.array_equal(bits(gpu_run(A, B, C)), bits(first))


def test_accumulates_across_calls():
    b, m, k, n = 2, 3, 128, 64
    A, B, C = w.make(b, m, k, n, seed=10, ab="int4", c="int8")
    once = oracle.matmul_accum(b, m, k, n, A, B, C)
    thrice = oracle.matmul_accum(b, m, k, n, A, B, oracle.matmul_accum(b, m, k, n, A, B, once))
    assert_bit_exact(gpu_run(A, B, C, calls=3), thrice, "three accumulating calls")


def test_back_to_back_calls_of_every_kernel_family_on_shared_buffers():
    """Calls are launched so that each may start while its predecessor drains; a chain that
    alternates kernel families on the same C (and re-uses one call's inputs in the next)
    must still equal the oracle applied in order.  Integer inputs: every call is exact."""
    b, k, n = 1, 512, 2048
    rows = [1, 16, 1, 160, 2, 40, 1, 300, 16, 1]          # GEMV, swapped, tiles, pairs, ...
    m_max = max(rows)
    A, B, C = w.make(b, m_max, k, n, seed=31, ab="int4", c="int8")
    B2 = w.make(b, 1, k, n, seed=32, ab="int4", c="zeros")[1]
    dA, dB, dC = to_dev(A, B, C)
    dB2 = torch.from_numpy(B2.view(np.int16)).cuda()
    want = C.copy()
    for step, m in enumerate(rows):
        Bs, dBs = (B, dB) if step % 2 == 0 else (B2, dB2)
        # rows [0, m) of A against C's first m rows: a sub-problem with the same row pitch
        mb.morello_matmul_accum(b, m, k, n, dA, dBs, dC)
        want[:, :m, :] = oracle.matmul_accum(b, m, k, n, np.ascontiguousarray(A[:, :m, :]), Bs,
                                             np.ascontiguousarray(want[:, :m, :]))
    st, detail = mb.morello_read_device_status()
    assert st == mb.MORELLO_OK, hex(detail)
    assert_bit_exact(dC.cpu().numpy(), want, "chain of calls on one C")


# ------------------------------------------------------------------ T5: guards
def test_canaries_around_c_stay_intact():
    b, m, k, n = 2, 5, 96, 40
    A, B, C = w.make(b, m, k, n, seed=11, ab="int4", c="normal")
    dA, dB, _ = to_dev(A, B, C)
    pad = 1024
    buf = torch.full((pad + C.size + pad,), 12345.0, device="cuda")
    buf[pad:pad + C.size] = torch.from_numpy(C.reshape(-1)).cuda()
    mb.morello_matmul_accum(b, m, k, n, dA, dB, buf[pad:])
    torch.cuda.synchronize()
    assert torch.all(buf[:pad] == 12345.0) and torch.all(buf[pad + C.size:] == 12345.0)
    assert_bit_exact(buf[pad:pad + C.size].cpu().numpy().reshape(b, m, n),
                     oracle.matmul_accum(b, m, k, n, A, B, C), "C between canaries")


def test_empty_shapes_launch_nothing():
    dA, dB, dC = to_dev(*w.make(1, 2, 4, 8, seed=1))
    before = dC.clone()
    launches = mb.morello_launch_count()
    for shape in [(0, 2, 4, 8), (1, 0, 4, 8), (1, 2, 0, 8), (1, 2, 4, 0)]:
        mb.morello_matmul_accum(*shape, dA, dB, dC)
    torch.cuda.synchronize()
    assert mb.morello_launch_count() == launches and torch.equal(before, dC)


def test_unaligned_operands_take_the_narrow_loads():
    b, m, k, n = 1, 3, 50, 24
    A, B, C = w.make(b, m, k, n, seed=12, ab="int4", c="int8")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    for off in (1, 2, 4):                # B starts 2, 4, 8 bytes past a 16-byte boundary
        big = torch.zeros(B.size + 8, dtype=torch.int16, device="cuda")
        big[off:off + B.size] = torch.from_numpy(B.view(np.int16).reshape(-1)).cuda()
        dA, _, dC = to_dev(A, B, C)
        mb.morello_matmul_accum(b, m, k, n, dA, big[off:], dC)
        assert_bit_exact(dC.cpu().numpy(), want, "B offset %d elements" % off)


def test_forced_tensor_path_refuses_shapes_it_cannot_address():
    b, m, k, n = 1, 64, 60, 36            # k, n not multiples of 8
    dA, dB, dC = to_dev(*w.make(b, m, k, n, seed=13))
    before = dC.clone()
    with pytest.raises(mb.MorelloError) as e:
        mb.morello_matmul_accum_forced(mb.MORELLO_PATH_TCGEN05, 0, b, m, k, n, dA, dB, dC)
    assert e.value.status == mb.MORELLO_ERR_UNSUPPORTED_PATH
    torch.cuda.synchronize()
    assert torch.equal(before, dC)


# ----------------------------------------------------- host-buffer entry point
def test_host_entry_point_round_trip():
    b, m, k, n = 2, 4, 256, 512
    A, B, C = w.make(b, m, k, n, seed=14, ab="int4", c="normal")
    want = oracle.matmul_accum(b, m, k, n, A, B, C)
    out = C.copy()
    mb.morello_matmul_accum_host(b, m, k, n, A, B, out)
    assert_bit_exact(out, want, "host entry point")
