"""The seeded generators: bf16 rounding, determinism, shapes and value ranges."""
import numpy as np

from paper_2505_01637_b200 import workloads as w


def test_bf16_rne_known_values():
    f = np.array([1.0, -2.0, 0.0, 1.00390625, 1.01171875, 3.140625], dtype=np.float32)
    h = w.f32_to_bf16_rne(f)
    # 1 + 2^-8 is a tie between 0x3F80 and 0x3F81 -> even; 1 + 3*2^-8 ties up to 0x3F82
    assert list(h) == [0x3F80, 0xC000, 0x0000, 0x3F80, 0x3F82, 0x4049]
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    back = w.bf16_to_f32(w.f32_to_bf16_rne(x))
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(w.f32_to_bf16_rne(back), w.f32_to_bf16_rne(x))  # idempotent


def test_configs_match_the_named_shapes():
    shapes = [c.shape for c in w.CONFIGS]
    assert shapes == [(1, 4, 4, 16), (1, 1, 2048, 16384), (1, 16, 2048, 16384),
                      (1, 4096, 4096, 4096), (8, 2048, 2048, 16384)]
    assert w.CONFIGS[1].algorithmic_bytes == 67_244_032
    assert w.CONFIGS[4].flops == 1_099_511_627_776


def test_generators_are_deterministic_and_in_range():
    A, B, C = w.make_config(0)
    A2, B2, C2 = w.make_config(0)
    assert w.crc32(A) == w.crc32(A2) and w.crc32(B) == w.crc32(B2) and w.crc32(C) == w.crc32(C2)
    assert np.abs(w.bf16_to_f32(A)).max() <= 1.0 and np.abs(w.bf16_to_f32(B)).max() <= 1.0
    Ai, Bi, Ci = w.make_config(0, "integer_intc")
    for t, lim in ((w.bf16_to_f32(Ai), 4), (w.bf16_to_f32(Bi), 4), (Ci, 8)):
        assert np.array_equal(t, np.round(t)) and np.abs(t).max() <= lim
    A3, B3, C3 = w.make(3, 2, 8, 4, seed=5)
    A1, B1, C1 = w.make(1, 2, 8, 4, seed=6)       # batch 1 of seed 5 == batch 0 of seed 6
    assert np.array_equal(A3[1], A1[0]) and np.array_equal(C3[1], C1[0])


def test_sample_rows():
    rows = w.sample_rows(8, 2048, seed=3)
    assert rows.min() == 0 and rows.max() < 8 * 2048 and len(np.unique(rows)) == len(rows)
    assert set(range(128)) <= set(rows) and set(range(1920, 2048)) <= set(rows)
    for beta in range(8):
        assert np.any((rows >= beta * 2048) & (rows < (beta + 1) * 2048))
