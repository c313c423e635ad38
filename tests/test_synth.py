"""Seeded input generators: determinism, ranges, packing and the sampling rule."""
import numpy as np

from paper_2608_10103_b200 import synth


def test_generators_are_deterministic_and_in_range():
    for prec in synth.PRECISIONS:
        A1, B1 = synth.make(prec, 40, 50, 64, seed=3)
        A2, B2 = synth.make(prec, 40, 50, 64, seed=3)
        assert np.array_equal(A1, A2) and np.array_equal(B1, B2)
        A3, _ = synth.make(prec, 40, 50, 64, seed=4)
        assert not np.array_equal(A1, A3)
    A, B = synth.fp16_uniform(64, 64, 256, 0)
    assert A.dtype == np.float16 and np.abs(A).max() <= 1.0
    A, B = synth.fp16_normal_clipped(64, 64, 256, 0)
    assert np.abs(A).max() <= 4.0 and np.abs(A).max() > 2.0
    A, B = synth.s8_uniform(64, 64, 512, 0)
    assert A.dtype == np.int8 and A.min() == -128 and A.max() == 127
    A, B = synth.s4_uniform(64, 64, 512, 0)
    assert A.dtype == np.uint8 and A.shape == (64, 256)
    lo, hi = A & 15, A >> 4
    assert set(np.unique(lo)) == set(range(16)) and set(np.unique(hi)) == set(range(16))


def test_pack_s4_byte_layout():
    v = np.array([[1, -1, 7, -8, 0, 5]])
    assert synth.pack_s4(v).tolist() == [[0xF1, 0x87, 0x50]]


def test_sweep_seeds_cover_10_to_24():
    seeds = [synth.sweep_seed(p, n) for p in synth.PRECISIONS for n in synth.SWEEP_SIZES]
    assert seeds == list(range(10, 25))


def test_sample_rows_cols():
    rows, cols = synth.sample_rows_cols(8192, 8192, seed=3)
    assert len(rows) >= 256 and len(cols) >= 256
    assert len(np.unique(rows)) == len(rows) and rows.min() >= 0 and rows.max() == 8191
    for edge in (0, 127, 128, 255, 256, 8191):
        assert edge in rows and edge in cols
    r2, c2 = synth.sample_rows_cols(8192, 8192, seed=3)
    assert np.array_equal(rows, r2) and np.array_equal(cols, c2)
    rows, cols = synth.sample_rows_cols(100, 300, seed=1)
    assert len(rows) == 100 and cols.max() == 299


def test_ops_convention():
    assert synth.gemm_ops(8192, 8192, 8192) == 2 * 8192 ** 3
