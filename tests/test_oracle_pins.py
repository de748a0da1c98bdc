"""Pins for the CPU oracle: it is checked against things other than itself --
exact rational arithmetic, hand arithmetic, closed forms, structural special
cases and integer / float64 library contractions -- chosen so that a dropped
term, a wrong sign or index, a transposed operand or a misplaced accumulate
fails at least one of them."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2505_01637_b200 import workloads as w

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- helpers
def frac_to_f32_bits(x: Fraction) -> int:
    """Exact rational -> IEEE binary32 bit pattern, round-to-nearest-even,
    written with integer arithmetic only (no float conversion involved)."""
    if x == 0:
        return 0
    sign = 0x80000000 if x < 0 else 0
    x = abs(x)
    e = x.numerator.bit_length() - x.denominator.bit_length()
    if Fraction(2) ** e > x:
        e -= 1                      # now 2^e <= x < 2^(e+1)
    e = max(e, -126)                # subnormals share the exponent of 2^-126
    q = x / (Fraction(2) ** (e - 23))   # significand in units of the last place
    fl = q.numerator // q.denominator
    rem = q - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (fl & 1)):
        fl += 1
    if fl >= (1 << 24):
        fl >>= 1
        e += 1
    assert e <= 127
    if fl < (1 << 23):              # subnormal
        return sign | fl
    return sign | ((e + 127) << 23) | (fl - (1 << 23))


def exact_matmul_accum_bits(A, B, C):
    b, m, k = A.shape
    n = B.shape[2]
    Af, Bf = w.bf16_to_f32(A), w.bf16_to_f32(B)
    out = np.zeros((b, m, n), dtype=np.uint32)
    for bb in range(b):
        for i in range(m):
            for j in range(n):
                s = Fraction(float(C[bb, i, j]))
                for p in range(k):
                    s += Fraction(float(Af[bb, i, p])) * Fraction(float(Bf[bb, p, j]))
                out[bb, i, j] = frac_to_f32_bits(s)
    return out


def as_bf16(x):
    h = w.f32_to_bf16_rne(np.asarray(x, dtype=np.float32))
    assert np.array_equal(w.bf16_to_f32(h), np.asarray(x, dtype=np.float32)), "not bf16-exact"
    return h


def run(A, B, C, naive=False):
    b, m, k = A.shape
    n = B.shape[2]
    return oracle.matmul_accum(b, m, k, n, A, B, C, naive=naive)


def bits(x):
    return np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)


# ------------------------------------------------- the rounding helper itself
def test_frac_to_f32_bits_known_values():
    assert frac_to_f32_bits(Fraction(1)) == 0x3F800000
    assert frac_to_f32_bits(Fraction(-2)) == 0xC0000000
    assert frac_to_f32_bits(Fraction(3, 2)) == 0x3FC00000
    # 1 + 2^-24 is a tie between 1 and 1 + 2^-23: goes to the even one (1)
    assert frac_to_f32_bits(1 + Fraction(1, 1 << 24)) == 0x3F800000
    # 1 + 3*2^-24 ties between 1+2^-23 (odd) and 1+2^-22 (even)
    assert frac_to_f32_bits(1 + Fraction(3, 1 << 24)) == 0x3F800002
    assert frac_to_f32_bits(1 + Fraction(1, 1 << 24) + Fraction(1, 1 << 40)) == 0x3F800001
    assert frac_to_f32_bits(Fraction(1, 1 << 149)) == 1           # smallest subnormal
    assert frac_to_f32_bits(Fraction(16777217)) == 0x4B800000     # 2^24 + 1 -> 2^24
    rng = np.random.default_rng(1)
    for v in rng.standard_normal(200).astype(np.float32):
        assert frac_to_f32_bits(Fraction(float(v))) == int(np.float32(v).view(np.uint32))


# ------------------------------------------------------ 1. exact brute force
@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (1, 4, 4, 16), (2, 3, 5, 7),
                                   (3, 2, 7, 9), (1, 5, 9, 3), (2, 1, 33, 5)])
@pytest.mark.parametrize("naive", [False, True])
def test_exact_rational_brute_force(shape, naive):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=11 + sum(shape), ab="uniform", c="normal")
    want = exact_matmul_accum_bits(A, B, C)
    got = run(A, B, C, naive=naive)
    assert np.array_equal(bits(got), want)


def test_figure1_config_exact():
    A, B, C = w.make_config(0)
    assert np.array_equal(bits(run(A, B, C)), exact_matmul_accum_bits(A, B, C))
    for variant in ("integer", "integer_intc"):
        A, B, C = w.make_config(0, variant)
        assert np.array_equal(bits(run(A, B, C)), exact_matmul_accum_bits(A, B, C))


# --------------------------------------------------------- hand-worked golden
def _read_golden(path):
    rec = {}
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            key, *vals = line.split()
            rec[key] = [float(v) for v in vals]
    return rec


def test_hand_worked_example():
    g = _read_golden(os.path.join(GOLDEN, "hand_worked_1x2x3x2.txt"))
    b, m, k, n = (int(v) for v in g["shape"])
    A = as_bf16(g["A"]).reshape(b, m, k)
    B = as_bf16(g["B"]).reshape(b, k, n)
    C = np.array(g["C"], dtype=np.float32).reshape(b, m, n)
    want = np.array(g["expect"], dtype=np.float32).reshape(b, m, n)
    for naive in (False, True):
        assert np.array_equal(run(A, B, C, naive=naive), want)


def test_cancelling_products_leave_c_to_the_last_bit():
    g = _read_golden(os.path.join(GOLDEN, "cancellation_1x1x2x1.txt"))
    b, m, k, n = (int(v) for v in g["shape"])
    A = as_bf16(g["A"]).reshape(b, m, k)
    B = as_bf16(g["B"]).reshape(b, k, n)
    C = np.array(g["C"], dtype=np.float32).reshape(b, m, n)
    want = np.array(g["expect"], dtype=np.float32).reshape(b, m, n)
    assert bits(want)[0, 0, 0] == 0x3F800001
    for naive in (False, True):
        assert np.array_equal(bits(run(A, B, C, naive=naive)), bits(want))
    assert np.array_equal(exact_matmul_accum_bits(A, B, C), bits(want))
    Bt = np.ascontiguousarray(np.swapaxes(B, 1, 2))
    assert np.array_equal(bits(oracle.matmul_accum_bt(b, m, k, n, A, Bt, C)), bits(want))
    assert np.array_equal(bits(oracle.matmul_accum_packed_b(1, b, m, k, n, A, w.pack_b(B, 1), C)), bits(want))
    got32 = oracle.matmul_accum_f32(b, m, k, n, w.bf16_to_f32(A), w.bf16_to_f32(B), C)
    assert np.array_equal(bits(got32), bits(want))
    # the arithmetic that starts the double sum from C does lose the bit: the pin sees it
    assert not np.array_equal(bits(_mutant(A, B, C, "c_first_double_sum")), bits(want))


def test_long_integer_sum_that_cancels_keeps_a_small_c_exactly():
    # One output element of a seeded 7 x 129 x 11175 x 104 problem with A, B integers in [-4, 4]:
    # its 11,175 products add up to zero while the partial sums reach into the hundreds, and C is
    # about 2^-21.  Exact rational arithmetic says the result is C; a double sum that starts from C
    # drops C's last bit on the way (it needs more than 53 bits there).
    A, B, C = w.make(7, 129, 11175, 104, seed=1300196, ab="int4", c="normal")
    a, bcol, c = A[4:5, 31:32, :], B[4:5, :, 87:88], C[4:5, 31:32, 87:88]
    a, bcol, c = np.ascontiguousarray(a), np.ascontiguousarray(bcol), np.ascontiguousarray(c)
    assert int((w.bf16_to_f32(a).astype(np.int64).reshape(-1) * w.bf16_to_f32(bcol).astype(np.int64).reshape(-1)).sum()) == 0
    want = exact_matmul_accum_bits(a, bcol, c)
    assert np.array_equal(want, bits(c))
    for naive in (False, True):
        assert np.array_equal(bits(run(a, bcol, c, naive=naive)), want)
    assert not np.array_equal(bits(_mutant(a, bcol, c, "c_first_double_sum")), want)


def _paper_shapes():
    out = []
    for line in open(os.path.join(GOLDEN, "paper_shapes.txt")):
        line = line.split("#")[0].strip()
        if line:
            out.append(tuple(int(v) for v in line.split()))
    return out


# ------------------------------------------------------------ 2. closed forms
@pytest.mark.parametrize("shape", _paper_shapes() + [(2, 3, 1000, 40)])
def test_closed_forms(shape):
    b, m, k, n = shape
    ones_a = as_bf16(np.ones((b, m, k)))
    ones_b = as_bf16(np.ones((b, k, n)))
    zero_c = np.zeros((b, m, n), dtype=np.float32)
    assert np.array_equal(run(ones_a, ones_b, zero_c), np.full((b, m, n), k, np.float32))
    colpat = (np.arange(n) % 8 - 4).astype(np.float32)
    Bc = as_bf16(np.broadcast_to(colpat, (b, k, n)).copy())
    assert np.array_equal(run(ones_a, Bc, zero_c),
                          np.broadcast_to(k * colpat, (b, m, n)))
    rowpat = (np.arange(m) % 5).astype(np.float32)
    Ar = as_bf16(np.broadcast_to(rowpat[:, None], (b, m, k)).copy())
    assert np.array_equal(run(Ar, ones_b, zero_c),
                          np.broadcast_to(k * rowpat[:, None], (b, m, n)))
    # alternating signs along k cancel in pairs: sum = (k odd)
    alt = np.where(np.arange(k) % 2 == 0, 1.0, -1.0).astype(np.float32)
    Aa = as_bf16(np.broadcast_to(alt, (b, m, k)).copy())
    assert np.array_equal(run(Aa, ones_b, zero_c), np.full((b, m, n), k % 2, np.float32))
    # weights along k: sum_p p  (pins that every p is visited once), p < 256 is bf16-exact
    kk = min(k, 256)
    ramp = np.zeros(k, np.float32)
    ramp[:kk] = np.arange(kk)
    Ap = as_bf16(np.broadcast_to(ramp, (b, m, k)).copy())
    assert np.array_equal(run(Ap, ones_b, zero_c),
                          np.full((b, m, n), kk * (kk - 1) // 2, np.float32))


# --------------------------------------- 3. identity / zero / one-hot operands
def _distinct_ints(shape, lo=-100, mod=201, seed=0):
    """Distinct-looking small integers (bf16-exact: |v| <= 128 after shift)."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, mod, size=shape) + lo).clip(-128, 128).astype(np.float32)


def test_identity_and_zero():
    b, d, n = 2, 6, 11
    Bv = _distinct_ints((b, d, n), seed=1)
    I = np.broadcast_to(np.eye(d, dtype=np.float32), (b, d, d)).copy()
    C = _distinct_ints((b, d, n), seed=2)
    assert np.array_equal(run(as_bf16(I), as_bf16(Bv), C), C + Bv)     # A = I  (m = k)
    Av = _distinct_ints((b, 5, d), seed=3)
    C2 = _distinct_ints((b, 5, d), seed=4)
    assert np.array_equal(run(as_bf16(Av), as_bf16(I), C2), C2 + Av)   # B = I  (k = n)
    Cr = np.random.default_rng(5).standard_normal((b, d, n)).astype(np.float32)
    Z = np.zeros((b, d, d), np.float32)
    assert np.array_equal(bits(run(as_bf16(Z), as_bf16(Bv), Cr)), bits(Cr))
    assert np.array_equal(bits(run(as_bf16(I), as_bf16(np.zeros((b, d, n))), Cr)), bits(Cr))


def test_one_hot_pins_layout():
    b, m, k, n = 3, 4, 5, 6
    Bv = _distinct_ints((b, k, n), seed=6)
    Av = _distinct_ints((b, m, k), seed=7)
    C = _distinct_ints((b, m, n), seed=8)
    for (b0, i0, p0) in [(0, 0, 0), (1, 2, 3), (2, 3, 4)]:
        A1 = np.zeros((b, m, k), np.float32)
        A1[b0, i0, p0] = 2.0
        want = C.copy()
        want[b0, i0, :] += 2.0 * Bv[b0, p0, :]
        assert np.array_equal(run(as_bf16(A1), as_bf16(Bv), C), want)
    for (b0, p0, j0) in [(0, 0, 0), (1, 3, 2), (2, 4, 5)]:
        B1 = np.zeros((b, k, n), np.float32)
        B1[b0, p0, j0] = -3.0
        want = C.copy()
        want[b0, :, j0] += -3.0 * Av[b0, :, p0]
        assert np.array_equal(run(as_bf16(Av), as_bf16(B1), C), want)


# ------------------------------------------------------ 4. accumulate invariant
def test_accumulate_invariant():
    b, m, k, n = 2, 5, 64, 24
    A, B, C = w.make(b, m, k, n, seed=21, ab="int4", c="int8")
    zero = np.zeros_like(C)
    assert np.array_equal(run(A, B, C), C + run(A, B, zero))
    # two accumulating calls = one call with the product doubled (integers: exact)
    twice = run(A, B, run(A, B, C))
    assert np.array_equal(twice, C + 2 * run(A, B, zero))
    # non-integer C with integer A, B: the exact sum rounded once
    _, _, Cn = w.make(b, m, k, n, seed=22, ab="int4", c="normal")
    prod = run(A, B, zero).astype(np.float64)
    assert np.array_equal(run(A, B, Cn), (Cn.astype(np.float64) + prod).astype(np.float32))


# -------------------------------------------------------- 5. integer exactness
@pytest.mark.parametrize("shape", [(1, 4, 4, 16), (2, 7, 130, 33), (1, 1, 2048, 96),
                                   (1, 16, 4096, 8)])
def test_integer_inputs_match_integer_matmul(shape):
    b, m, k, n = shape
    A, B, C = w.make(b, m, k, n, seed=31, ab="int4", c="int8")
    Ai = w.bf16_to_f32(A).astype(np.int64)
    Bi = w.bf16_to_f32(B).astype(np.int64)
    want = (C.astype(np.int64) + np.matmul(Ai, Bi)).astype(np.float32)
    assert np.abs(np.matmul(Ai, Bi)).max() < 2 ** 24
    assert np.array_equal(run(A, B, C), want)


# ------------------------------------------------------- 6. power-of-two scaling
def test_power_of_two_scaling_is_exact():
    b, m, k, n = 1, 3, 50, 20
    A, B, C = w.make(b, m, k, n, seed=41, ab="uniform", c="zeros")
    base = run(A, B, C)
    A8 = w.f32_to_bf16_rne(w.bf16_to_f32(A) * np.float32(8.0))
    B4 = w.f32_to_bf16_rne(w.bf16_to_f32(B) * np.float32(0.25))
    assert np.array_equal(run(A8, B, C), base * np.float32(8.0))
    assert np.array_equal(run(A, B4, C), base * np.float32(0.25))
    An = w.f32_to_bf16_rne(-w.bf16_to_f32(A))
    assert np.array_equal(run(An, B, C), -base)


# ------------------------------------------------ 7. float64 library contraction
@pytest.mark.parametrize("cfg", [("uniform", "normal"), ("normal_rsqrtk", "normal0.1")])
def test_agrees_with_float64_matmul(cfg):
    b, m, k, n = 2, 9, 300, 70
    A, B, C = w.make(b, m, k, n, seed=51, ab=cfg[0], c=cfg[1])
    ref64 = C.astype(np.float64) + np.matmul(w.bf16_to_f32(A).astype(np.float64),
                                             w.bf16_to_f32(B).astype(np.float64))
    got = run(A, B, C)
    ulp = np.spacing(np.abs(ref64).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(got.astype(np.float64) - ref64) <= 0.5000001 * ulp + 1e-300)


# ------------------------------------------------------------ 8. host plumbing
def test_rows_and_abs_dot_helpers():
    b, m, k, n = 3, 10, 40, 17
    A, B, C = w.make(b, m, k, n, seed=61)
    full = run(A, B, C)
    rows = np.array([0, 9, 10, 17, 29], dtype=np.int64)
    out, T = oracle.matmul_accum_rows(b, m, k, n, A, B, C, rows)
    assert np.array_equal(bits(out), bits(full.reshape(b * m, n)[rows]))
    Tref = np.matmul(np.abs(w.bf16_to_f32(A).astype(np.float64)),
                     np.abs(w.bf16_to_f32(B).astype(np.float64)))
    assert np.allclose(T, Tref.reshape(b * m, n)[rows], rtol=1e-13, atol=0)
    assert np.allclose(oracle.abs_dot(b, m, k, n, A, B), Tref, rtol=1e-13, atol=0)


def test_empty_shapes():
    for shape in [(0, 3, 4, 5), (2, 0, 4, 5), (2, 3, 4, 0)]:
        b, m, k, n = shape
        A, B, C = w.make(b, m, k, n, seed=1)
        assert run(A, B, C).shape == (b, m, n)
    A, B, C = w.make(2, 3, 0, 5, seed=1)          # empty sum: C unchanged
    assert np.array_equal(bits(run(A, B, C)), bits(C))


# ------------------------------------- 9. the pins catch planted mistakes (CPU)
def _mutant(A, B, C, kind):
    """A float64 restatement of the definition with one planted mistake."""
    Af = w.bf16_to_f32(A).astype(np.float64)
    Bf = w.bf16_to_f32(B).astype(np.float64)
    Cd = C.astype(np.float64)
    if kind == "drop_last_term":
        return (Cd + np.matmul(Af[:, :, :-1], Bf[:, :-1, :])).astype(np.float32)
    if kind == "no_accumulate":
        return np.matmul(Af, Bf).astype(np.float32)
    if kind == "wrong_sign":
        return (Cd - np.matmul(Af, Bf)).astype(np.float32)
    if kind == "batch0_operand":
        return (Cd + np.matmul(Af, Bf[:1])).astype(np.float32)
    if kind == "transposed_b":
        return (Cd + np.matmul(Af, np.swapaxes(Bf, 1, 2))).astype(np.float32)
    if kind == "c_first_double_sum":   # a double sum that starts from C can lose C's low bits
        s = Cd.copy()
        for p in range(Af.shape[2]):
            s = s + Af[:, :, p:p + 1] * Bf[:, p:p + 1, :]
        return s.astype(np.float32)
    if kind == "f32_preload_sum":   # accumulating in f32 from C is a different rounding
        s = C.copy()
        for p in range(Af.shape[2]):
            s = (s + (Af[:, :, p:p + 1] * Bf[:, p:p + 1, :]).astype(np.float32)).astype(np.float32)
        return s
    raise ValueError(kind)


@pytest.mark.parametrize("kind", ["drop_last_term", "no_accumulate", "wrong_sign",
                                  "batch0_operand", "transposed_b", "f32_preload_sum"])
def test_pins_detect_planted_mistakes(kind):
    b, d = 2, 6                      # square so the transposed mutant type-checks
    A, B, C = w.make(b, d, d, d, seed=71, ab="uniform", c="normal")
    if kind == "f32_preload_sum":
        A, B, C = w.make(1, 4, 512, 16, seed=72, ab="uniform", c="normal")
    want = exact_matmul_accum_bits(A, B, C)
    assert np.array_equal(bits(run(A, B, C)), want)
    assert not np.array_equal(bits(_mutant(A, B, C, kind)), want)


# ---------------------------------------------------- float32-input oracle (Section 7's
# float32 2048-square matmul): pinned to the bf16 oracle above, to exact rational
# arithmetic and to layout one-hots
def exact_f32_bits(A, B, C):
    b, m, k = A.shape
    n = B.shape[2]
    out = np.zeros((b, m, n), dtype=np.uint32)
    for bb in range(b):
        for i in range(m):
            for j in range(n):
                s = Fraction(float(C[bb, i, j]))
                for p in range(k):
                    s += Fraction(float(A[bb, i, p])) * Fraction(float(B[bb, p, j]))
                out[bb, i, j] = frac_to_f32_bits(s)
    return out


def test_f32_oracle_equals_bf16_oracle_on_bf16_representable_inputs():
    for (b, m, k, n) in [(1, 4, 4, 16), (2, 3, 65, 40), (1, 1, 257, 33)]:
        A, B, C = w.make(b, m, k, n, seed=3 + k, ab="uniform", c="normal")
        want = oracle.matmul_accum(b, m, k, n, A, B, C)
        got = oracle.matmul_accum_f32(b, m, k, n, w.bf16_to_f32(A), w.bf16_to_f32(B), C)
        assert np.array_equal(bits(got), bits(want))


@pytest.mark.parametrize("shape", [(1, 1, 1, 1), (2, 3, 5, 7), (1, 4, 9, 3)])
def test_f32_oracle_exact_rational_brute_force(shape):
    b, m, k, n = shape
    rng = np.random.Generator(np.random.Philox(40 + sum(shape)))
    # 12 significant bits per input: products have 24, and sums of a few of them are exact in
    # double, so the oracle's single rounding must equal the exact result's rounding
    def q12(x):
        mant, ex = np.frexp(x.astype(np.float64))
        return np.ldexp(np.round(mant * 4096) / 4096, ex).astype(np.float32)
    A = q12(rng.standard_normal((b, m, k)))
    B = q12(rng.standard_normal((b, k, n)))
    C = q12(rng.standard_normal((b, m, n)))
    got = oracle.matmul_accum_f32(b, m, k, n, A, B, C)
    assert np.array_equal(bits(got), exact_f32_bits(A, B, C))
    # full-precision inputs: the double sum may round once more than the exact one; never
    # further than one unit in the last place
    A = rng.standard_normal((b, m, k)).astype(np.float32)
    B = rng.standard_normal((b, k, n)).astype(np.float32)
    C = rng.standard_normal((b, m, n)).astype(np.float32)
    got = bits(oracle.matmul_accum_f32(b, m, k, n, A, B, C)).astype(np.int64)
    want = exact_f32_bits(A, B, C).astype(np.int64)
    assert np.abs(got - want).max() <= 1


def test_f32_oracle_one_hot_layout_abs_dot_and_float64_agreement():
    b, m, k, n = 3, 4, 6, 5
    rng = np.random.default_rng(5)
    Bv = rng.integers(-100, 101, size=(b, k, n)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    A1 = np.zeros((b, m, k), np.float32)
    A1[1, 2, 4] = 2.0
    want = C.copy()
    want[1, 2, :] += 2.0 * Bv[1, 4, :]
    assert np.array_equal(oracle.matmul_accum_f32(b, m, k, n, A1, Bv, C), want)
    A = rng.standard_normal((b, m, k)).astype(np.float32)
    B = rng.standard_normal((b, k, n)).astype(np.float32)
    got, T = oracle.matmul_accum_f32(b, m, k, n, A, B, C, want_abs=True)
    ref = C.astype(np.float64) + np.einsum("bik,bkj->bij", A.astype(np.float64), B.astype(np.float64))
    assert np.abs(got - ref).max() <= np.spacing(np.abs(ref).max().astype(np.float32))
    assert np.allclose(T, np.einsum("bik,bkj->bij", np.abs(A).astype(np.float64), np.abs(B).astype(np.float64)), rtol=1e-12)


# ------------------------------------------------ column-major right-hand side (Section 2.2's
# Spec example has a col_major rhs): pinned to the row-major oracle and to a one-hot
def test_colmajor_oracle_equals_rowmajor_oracle_on_the_transposed_operand():
    for (b, m, k, n) in [(1, 4, 128, 16), (2, 3, 65, 40), (3, 1, 7, 9)]:      # first: the Spec example's shape
        A, B, C = w.make(b, m, k, n, seed=21 + k, ab="uniform", c="normal")
        Bt = np.ascontiguousarray(B.transpose(0, 2, 1))
        assert np.array_equal(bits(oracle.matmul_accum_bt(b, m, k, n, A, Bt, C)),
                              bits(oracle.matmul_accum(b, m, k, n, A, B, C)))


def test_colmajor_oracle_one_hot_pins_the_indexing():
    b, m, k, n = 2, 3, 5, 4
    rng = np.random.default_rng(9)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    Bt1 = np.zeros((b, n, k), np.float32)
    Bt1[1, 2, 3] = -3.0                                  # B[1][p=3][j=2]
    want = C.copy()
    want[1, :, 2] += -3.0 * Av[1, :, 3]
    got = oracle.matmul_accum_bt(b, m, k, n, as_bf16(Av), as_bf16(Bt1), C)
    assert np.array_equal(got, want)


# ------------------------------------------------ packed right-hand side (Section 2.4.2: a strip
# dimension of size s on the column index): pinned to the offset formula written out, to a
# hand-computed offset, and to the row-major oracle
def test_packed_oracle_follows_the_offset_formula():
    for (s, b, m, k, n) in [(4, 2, 3, 5, 10), (8, 1, 2, 7, 8), (64, 1, 2, 3, 70), (16, 3, 1, 9, 5)]:
        A, B, C = w.make(b, m, k, n, seed=31 + s, ab="uniform", c="normal")
        strips = (n + s - 1) // s
        Bp = np.full(b * strips * k * s, 0x7FC0, np.uint16)          # padding = NaN patterns: never read
        for bb in range(b):
            for p in range(k):
                for j in range(n):
                    Bp[bb * strips * k * s + (j // s) * k * s + p * s + (j % s)] = B[bb, p, j]
        got = oracle.matmul_accum_packed_b(s, b, m, k, n, A, Bp, C)
        assert np.array_equal(bits(got), bits(oracle.matmul_accum(b, m, k, n, A, B, C)))
        assert np.array_equal(w.pack_b(B, s, fill=0x7FC0).reshape(-1), Bp)   # the test helper packs the same way


def test_packed_oracle_one_hot_at_a_hand_computed_offset():
    s, b, m, k, n = 4, 1, 3, 5, 10                       # 3 strips of 4 columns, 5 rows each
    rng = np.random.default_rng(11)
    Av = rng.integers(-100, 101, size=(b, m, k)).astype(np.float32)
    C = rng.integers(-50, 51, size=(b, m, n)).astype(np.float32)
    Bp = np.zeros(3 * 5 * 4, np.float32)
    Bp[1 * 20 + 3 * 4 + 2] = -3.0                        # strip 1, row p = 3, column 2 of the strip: j = 6
    want = C.copy()
    want[0, :, 6] += -3.0 * Av[0, :, 3]
    got = oracle.matmul_accum_packed_b(s, b, m, k, n, as_bf16(Av), as_bf16(Bp), C)
    assert np.array_equal(got, want)


# ------------------------------------------------- IEEE special values
def special_expectation(A, B, C, kinds):
    """What IEEE 754 arithmetic fixes for the planted inputs, written out by hand: per element
    either ("bits", pattern) or ("nan",)."""
    m, k = A.shape[1], A.shape[2]
    n = B.shape[2]
    Ai = w.bf16_to_f32(A)[0].astype(np.float64)
    Bi = w.bf16_to_f32(B)[0].astype(np.float64)
    POS_INF, NEG_INF = 0x7F800000, 0xFF800000
    out = {}
    for i in range(m):
        for j in range(n):
            kind = kinds[i]
            if kind == "ordinary":
                if j == 6:                         # 1 x (+Inf) joins finite terms
                    out[i, j] = ("bits", POS_INF)
                else:                              # integers only: k indices 0-4 of A are zero
                    total = int(C[0, i, j]) + sum(int(Ai[i, p]) * int(Bi[p, j]) for p in range(5, k))
                    out[i, j] = ("bits", frac_to_f32_bits(Fraction(total)))
            elif j == 6:                           # a special row has a zero against B's +Inf
                out[i, j] = ("nan",)
            elif kind == "subnormal_input":        # 2^-133 x 2^100
                out[i, j] = ("bits", frac_to_f32_bits(Fraction(1, 1 << 33)))
            elif kind == "subnormal_product":      # 2^-70 x 2^-70: a subnormal float32
                out[i, j] = ("bits", 1 << 9)
            elif kind == "pos_inf":                # Inf x 1, but Inf x 0 in column 5
                out[i, j] = ("nan",) if j == 5 else ("bits", POS_INF)
            elif kind == "neg_inf":                # -Inf x 1
                out[i, j] = ("bits", NEG_INF)
            else:                                  # a NaN operand; Inf - Inf
                out[i, j] = ("nan",)
    return out


@pytest.mark.parametrize("first", [0, 3])
def test_special_values_follow_ieee(first):
    m, k, n = 9, 12, 10
    A, B, C, kinds = w.make_special(m, k, n, seed=97, first=first)
    assert set(kinds[:6]) == set(w.SPECIAL_KINDS) and kinds[6:] == ["ordinary"] * 3
    want = special_expectation(A, B, C, kinds)
    Bt = np.ascontiguousarray(np.swapaxes(B, 1, 2))
    Af, Bf = w.bf16_to_f32(A), w.bf16_to_f32(B)
    results = {
        "row buffered": oracle.matmul_accum(1, m, k, n, A, B, C),
        "naive": oracle.matmul_accum(1, m, k, n, A, B, C, naive=True),
        "column-major B": oracle.matmul_accum_bt(1, m, k, n, A, Bt, C),
        "packed B": oracle.matmul_accum_packed_b(4, 1, m, k, n, A, w.pack_b(B, 4), C),
        "float32 inputs": oracle.matmul_accum_f32(1, m, k, n, Af, Bf, C),
    }
    for name, got in results.items():
        gb = bits(got)[0]
        for (i, j), e in want.items():
            if e[0] == "nan":
                assert np.isnan(got[0, i, j]), (name, kinds[i], i, j, got[0, i, j])
            else:
                assert int(gb[i, j]) == e[1], (name, kinds[i], i, j, hex(int(gb[i, j])), hex(e[1]))
