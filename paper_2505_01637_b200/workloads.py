"""Seeded synthetic inputs for MatmulAccum.

This module holds data generation only -- none of the method's arithmetic --
so that the CPU oracle's tests and the CUDA path's tests can both draw the
same tensors from it.  It imports numpy and nothing else from this project.

The paper's workloads are dense matrix multiplies with no dataset: the shapes
are the ones it names (Figure 1: b,m,k,n = 1,4,4,16; Section 7: the
1 x 2048 x 16384 bf16 -> f32 vector-matrix multiply), widened with a skinny
decode-style batch, a square GEMM and a large batched GEMM.  Its gemma.cpp
integration used model weights; the tensors drawn here stand in for them.

Recipe: ``rng = numpy.random.Generator(numpy.random.Philox(seed))`` with
``seed = 1000 * c + beta`` for config index c (0-based) and batch beta; A[beta],
then B[beta], then C[beta] are drawn in that order, row-major, as f32; A and B
are then rounded once to bf16 (round-to-nearest-even, integer arithmetic on the
f32 bit pattern).  Integer variants use ``seed + 500``.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    b: int
    m: int
    k: int
    n: int
    ab: str          # distribution of A and B: "uniform", "uniform_rsqrtk", "normal_rsqrtk"
    c: str           # distribution of C: "zeros", "normal", "normal0.1"
    note: str

    @property
    def shape(self):
        return (self.b, self.m, self.k, self.n)

    @property
    def macs(self):
        return self.b * self.m * self.k * self.n

    @property
    def flops(self):
        return 2 * self.macs

    @property
    def algorithmic_bytes(self):
        """A and B read once, C read once and written once."""
        b, m, k, n = self.shape
        return 2 * b * m * k + 2 * b * k * n + 2 * 4 * b * m * n


CONFIGS = (
    Config("cfg1_figure1", 1, 4, 4, 16, "uniform", "normal",
           "Figure 1 shape"),
    Config("cfg2_gemv", 1, 1, 2048, 16384, "uniform", "zeros",
           "Section 7 vector-matrix multiply, HBM-bound"),
    Config("cfg3_skinny16", 1, 16, 2048, 16384, "uniform_rsqrtk", "normal",
           "decode-style batch, GEMV/GEMM crossover"),
    Config("cfg4_square4096", 1, 4096, 4096, 4096, "normal_rsqrtk", "zeros",
           "square GEMM, tensor-core bound"),
    Config("cfg5_batched", 8, 2048, 2048, 16384, "normal_rsqrtk", "normal0.1",
           "large batched GEMM with fused accumulate epilogue"),
)


def f32_to_bf16_rne(x: np.ndarray) -> np.ndarray:
    """Round f32 to bf16 bit patterns (uint16), ties to even; finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(h: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to f32 exactly."""
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32)
            << np.uint32(16)).view(np.float32)


def _draw_ab(rng, shape, dist, k):
    if dist == "uniform":
        x = rng.random(shape, dtype=np.float32) * np.float32(2) - np.float32(1)
    elif dist == "uniform_rsqrtk":
        x = rng.random(shape, dtype=np.float32) * np.float32(2) - np.float32(1)
        x *= np.float32(1.0 / np.sqrt(k))
    elif dist == "normal_rsqrtk":
        x = rng.standard_normal(shape, dtype=np.float32)
        x *= np.float32(1.0 / np.sqrt(k))
    elif dist == "int4":
        x = rng.integers(-4, 5, size=shape).astype(np.float32)
    else:
        raise ValueError(dist)
    return f32_to_bf16_rne(x)


def _draw_c(rng, shape, dist):
    if dist == "zeros":
        return np.zeros(shape, dtype=np.float32)
    if dist == "normal":
        return rng.standard_normal(shape, dtype=np.float32)
    if dist == "normal0.1":
        return rng.standard_normal(shape, dtype=np.float32) * np.float32(0.1)
    if dist == "int8":
        return rng.integers(-8, 9, size=shape).astype(np.float32)
    raise ValueError(dist)


def make(b, m, k, n, seed, ab="uniform", c="normal"):
    """(A, B, C) for an arbitrary shape: A, B uint16 bf16 patterns, C f32.

    Batch beta is drawn from Philox(seed + beta): A, then B, then C."""
    A = np.empty((b, m, k), dtype=np.uint16)
    B = np.empty((b, k, n), dtype=np.uint16)
    C = np.empty((b, m, n), dtype=np.float32)
    for beta in range(b):
        rng = np.random.Generator(np.random.Philox(seed + beta))
        A[beta] = _draw_ab(rng, (m, k), ab, max(k, 1))
        B[beta] = _draw_ab(rng, (k, n), ab, max(k, 1))
        C[beta] = _draw_c(rng, (m, n), c)
    return A, B, C


def make_config(index: int, variant: str = "random"):
    """Inputs of benchmark configuration ``index`` (0-based).

    variant: "random" (the config's own distributions), "integer" (A, B integer
    uniform in [-4, 4], C as the config says) or "integer_intc" (C integers in
    [-8, 8] as well)."""
    cfg = CONFIGS[index]
    b, m, k, n = cfg.shape
    if variant == "random":
        return make(b, m, k, n, 1000 * index, cfg.ab, cfg.c)
    if variant == "integer":
        return make(b, m, k, n, 1000 * index + 500, "int4", cfg.c)
    if variant == "integer_intc":
        return make(b, m, k, n, 1000 * index + 500, "int4", "int8")
    raise ValueError(variant)


SPECIAL_KINDS = ("subnormal_input", "subnormal_product", "pos_inf", "nan", "inf_minus_inf", "neg_inf")

BF16_MIN_SUBNORMAL = 0x0001     # 2^-133
BF16_TWO_POW_100 = 0x7180
BF16_TWO_POW_MINUS_70 = 0x1C80
BF16_ONE = 0x3F80
BF16_POS_INF = 0x7F80
BF16_NEG_INF = 0xFF80
BF16_QUIET_NAN = 0x7FC0


def make_special(m, k, n, seed, first=0):
    """One batch with IEEE special values planted among small integers (k >= 8, n >= 8).

    Rows 0-5 of B are fixed: row 0 = 2^100, row 1 = 2^-70, row 2 = 1 except a 0 in column 5,
    row 4 = 1, row 5 = its integers except +Inf in column 6 (row 3 keeps its integers).  Row i of A,
    for i < 6, is zero but for what its kind plants (kind = SPECIAL_KINDS[(i + first) % 6]):
    the smallest bf16 subnormal at k index 0; 2^-70 at index 1; +Inf at 2; a NaN at 3; +Inf at 2
    and -Inf at 4; -Inf at 4.  Those rows start from C = 0.  Every later row is ordinary: integers
    with zeros at k indices 0-4 and a 1 at index 5 (so that it meets B's +Inf with a factor of 1).
    Returns (A, B, C, kinds) with kinds[i] the row's kind or "ordinary"."""
    assert k >= 8 and n >= 8
    A, B, C = make(1, m, k, n, seed, ab="int4", c="int8")
    A[0, :, 0:5] = 0
    A[0, :, 5] = BF16_ONE
    B[0, 0, :] = BF16_TWO_POW_100
    B[0, 1, :] = BF16_TWO_POW_MINUS_70
    B[0, 2, :] = BF16_ONE
    B[0, 2, 5] = 0
    B[0, 4, :] = BF16_ONE
    B[0, 5, 6] = BF16_POS_INF
    kinds = ["ordinary"] * m
    for i in range(min(m, len(SPECIAL_KINDS))):
        kind = SPECIAL_KINDS[(i + first) % len(SPECIAL_KINDS)]
        kinds[i] = kind
        A[0, i, :] = 0
        C[0, i, :] = 0
        if kind == "subnormal_input":
            A[0, i, 0] = BF16_MIN_SUBNORMAL
        elif kind == "subnormal_product":
            A[0, i, 1] = BF16_TWO_POW_MINUS_70
        elif kind == "pos_inf":
            A[0, i, 2] = BF16_POS_INF
        elif kind == "nan":
            A[0, i, 3] = BF16_QUIET_NAN
        elif kind == "inf_minus_inf":
            A[0, i, 2] = BF16_POS_INF
            A[0, i, 4] = BF16_NEG_INF
        elif kind == "neg_inf":
            A[0, i, 4] = BF16_NEG_INF
    return A, B, C, kinds


def crc32(x: np.ndarray) -> int:
    return zlib.crc32(np.ascontiguousarray(x).view(np.uint8).reshape(-1).data) & 0xFFFFFFFF


def sample_rows(b, m, seed, edge=128, stride=64):
    """Flattened row ids (bb*m + i) for sampled checks of a large problem: the
    first and last ``edge`` rows of batch 0 plus, in every batch, one seeded
    random row out of each block of ``stride`` rows (sorted, unique)."""
    rng = np.random.Generator(np.random.Philox(seed))
    rows = set(range(min(edge, m))) | set(range(max(0, m - edge), m))
    for beta in range(b):
        for i0 in range(0, m, stride):
            rows.add(beta * m + i0 + int(rng.integers(0, min(stride, m - i0))))
    return np.array(sorted(rows), dtype=np.int64)


def pack_b(B: np.ndarray, strip: int, fill: int = 0) -> np.ndarray:
    """B[b][k][n] (any 16-bit patterns) -> the packed layout Bp[b][ceil(n/strip)][k][strip]:
    strips of `strip` columns, row-major inside a strip, the last strip padded with `fill`."""
    b, k, n = B.shape
    strips = (n + strip - 1) // strip
    padded = np.full((b, k, strips * strip), fill, dtype=B.dtype)
    padded[:, :, :n] = B
    return np.ascontiguousarray(padded.reshape(b, k, strips, strip).transpose(0, 2, 1, 3))
