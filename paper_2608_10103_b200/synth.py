"""Seeded synthetic GEMM inputs (host side, numpy only).

This module only draws and packs bytes; it contains none of the GEMM
arithmetic.  The arrays it returns are the single source of truth handed to
both the CUDA library and the CPU checker.

The study this library follows runs square sizes N in {512 ... 8192} and does
not state value distributions (Sec. III-B), so the distributions here are the
ones the benchmark configuration names: uniform [-1, 1] or clipped N(0, 1) for
FP16, uniform integers over the full signed range for INT8 and INT4.
"""
from __future__ import annotations

import numpy as np

PRECISIONS = ("fp16", "s8", "s4")
SWEEP_SIZES = (512, 1024, 2048, 4096, 8192)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def pack_s4(values: np.ndarray) -> np.ndarray:
    """(R, K) integers in [-8, 7] -> (R, K/2) uint8, element 2m in the low
    nibble of byte m and element 2m+1 in the high nibble (two's complement)."""
    v = np.asarray(values)
    assert v.ndim == 2 and v.shape[1] % 2 == 0
    assert v.min(initial=0) >= -8 and v.max(initial=0) <= 7
    n = (v.astype(np.int16) & 15).astype(np.uint8)
    return (n[:, 0::2] | (n[:, 1::2] << 4)).astype(np.uint8)


def fp16_uniform(M: int, N: int, K: int, seed: int):
    """A (M,K), B (N,K): float64 uniform(-1, 1) rounded to nearest-even fp16.
    A is drawn first, then B, from one generator."""
    g = _rng(seed)
    A = g.uniform(-1.0, 1.0, size=(M, K)).astype(np.float16)
    B = g.uniform(-1.0, 1.0, size=(N, K)).astype(np.float16)
    return A, B


def fp16_normal_clipped(M: int, N: int, K: int, seed: int):
    """A, B ~ N(0,1) saturated to [-4, 4], then rounded to fp16."""
    g = _rng(seed)
    A = np.clip(g.standard_normal(size=(M, K)), -4.0, 4.0).astype(np.float16)
    B = np.clip(g.standard_normal(size=(N, K)), -4.0, 4.0).astype(np.float16)
    return A, B


def s8_uniform(M: int, N: int, K: int, seed: int):
    """A, B int8 uniform over [-128, 127]."""
    g = _rng(seed)
    A = g.integers(-128, 128, size=(M, K), dtype=np.int8)
    B = g.integers(-128, 128, size=(N, K), dtype=np.int8)
    return A, B


def s4_uniform(M: int, N: int, K: int, seed: int):
    """A, B signed 4-bit uniform over [-8, 7], packed (see pack_s4)."""
    g = _rng(seed)
    A = g.integers(-8, 8, size=(M, K), dtype=np.int8)
    B = g.integers(-8, 8, size=(N, K), dtype=np.int8)
    return pack_s4(A), pack_s4(B)


def make(precision: str, M: int, N: int, K: int, seed: int, dist: str = "uniform"):
    if precision == "fp16":
        if dist == "normal_clipped":
            return fp16_normal_clipped(M, N, K, seed)
        return fp16_uniform(M, N, K, seed)
    if precision == "s8":
        return s8_uniform(M, N, K, seed)
    if precision == "s4":
        return s4_uniform(M, N, K, seed)
    raise ValueError("unknown precision %r" % (precision,))


def sweep_seed(precision: str, N: int) -> int:
    """Seeds 10..24 of the precision x size sweep: 10 + 5*p + index of N."""
    return 10 + 5 * PRECISIONS.index(precision) + SWEEP_SIZES.index(N)


def sample_rows_cols(M: int, N: int, seed: int, count: int = 256):
    """Rows and columns checked at sizes too large for a full CPU compare:
    `count` distinct random rows and columns plus the tile-edge indices
    {0, 127, 128, 255, 256, last}."""
    g = _rng(seed + 1000)
    rows = g.choice(M, size=min(count, M), replace=False)
    cols = g.choice(N, size=min(count, N), replace=False)
    edge = np.array([0, 127, 128, 255, 256])
    rows = np.unique(np.concatenate([rows, edge[edge < M], [M - 1]]))
    cols = np.unique(np.concatenate([cols, edge[edge < N], [N - 1]]))
    return rows.astype(np.int32), cols.astype(np.int32)


def gemm_ops(M: int, N: int, K: int) -> int:
    """Operation count convention of the study's throughput tables
    (Table II: TOPS = 2 N^3 / duration): one multiply-accumulate = 2 ops."""
    return 2 * M * N * K
