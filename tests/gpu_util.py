"""Shared helpers for the GPU parity tests (host<->device plumbing only)."""
import numpy as np
import torch

import oracle
from paper_2608_10103_b200 import binding, synth

FULL_COMPARE_MAX = 2048


def to_dev(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def run_gpu(prec: str, A: np.ndarray, B: np.ndarray, fill=None) -> np.ndarray:
    """One call through the C-ABI; C is pre-filled with `fill` when given so a
    missed store shows up."""
    dA, dB = to_dev(A), to_dev(B)
    M, N = A.shape[0], B.shape[0]
    dtype = torch.float32 if prec == "fp16" else torch.int32
    C = torch.empty((M, N), dtype=dtype, device="cuda")
    if fill is not None:
        C.fill_(fill)
    binding.gemm(prec, dA, dB, C)
    torch.cuda.synchronize()
    return C.cpu().numpy()


def oracle_block(prec, A, B, rows=None, cols=None):
    """(C_ref, S) for the requested block; S is None for the integer paths."""
    if prec == "fp16":
        return oracle.gemm_fp16(A, B, rows, cols)
    if prec == "s8":
        return oracle.gemm_s8(A, B, rows, cols), None
    return oracle.gemm_s4(A, B, 2 * A.shape[1], rows, cols), None


def assert_block(prec, got, ref, S, what):
    if prec == "fp16":
        ok, worst = oracle.fp16_check(got, ref, S)
        assert ok, "%s: fp16 error %.3g x bound" % (what, worst)
    else:
        assert got.dtype == np.int32
        if not np.array_equal(got, ref):
            bad = np.argwhere(got != ref)
            i, j = bad[0]
            raise AssertionError("%s: %d mismatches, first at (%d,%d): got %d want %d" % (
                what, len(bad), i, j, got[i, j], ref[i, j]))


def check_against_oracle(prec, A, B, C, seed=0, force_full=False):
    """Full compare for small problems; 256 random rows + 256 random columns
    (plus tile-edge rows/columns) above FULL_COMPARE_MAX."""
    M, N = A.shape[0], B.shape[0]
    if force_full or max(M, N) <= FULL_COMPARE_MAX:
        ref, S = oracle_block(prec, A, B)
        assert_block(prec, C, ref, S, "full")
        return M * N
    rows, cols = synth.sample_rows_cols(M, N, seed)
    ref, S = oracle_block(prec, A, B, rows=rows)
    assert_block(prec, C[rows], ref, S, "rows")
    ref, S = oracle_block(prec, A, B, cols=cols)
    assert_block(prec, C[:, cols], ref, S, "cols")
    return len(rows) * N + len(cols) * M


def decode_s4(P: np.ndarray) -> np.ndarray:
    """Test-side nibble decoder (numpy)."""
    lo = (P & 0x0F).astype(np.int16)
    hi = (P >> 4).astype(np.int16)
    out = np.empty((P.shape[0], 2 * P.shape[1]), dtype=np.int16)
    out[:, 0::2] = np.where(lo >= 8, lo - 16, lo)
    out[:, 1::2] = np.where(hi >= 8, hi - 16, hi)
    return out


def freivalds(prec, A, B, C, seed, vectors=8):
    """Whole-matrix probabilistic check: C x == A (B^T x) for random x in
    {-1,0,1}^N.  Exact in int64 for the integer paths."""
    g = np.random.Generator(np.random.PCG64(seed))
    if prec == "s4":
        a = decode_s4(A).astype(np.int64)
        b = decode_s4(B).astype(np.int64)
    elif prec == "s8":
        a, b = A.astype(np.int64), B.astype(np.int64)
    else:
        a, b = A.astype(np.float64), B.astype(np.float64)
    X = g.integers(-1, 2, size=(B.shape[0], vectors))
    if prec == "fp16":
        X = X.astype(np.float64)
        lhs = C.astype(np.float64) @ X
        rhs = a @ (b.T @ X)
        bound = (np.abs(a) @ (np.abs(b.T) @ np.abs(X))) * oracle.FP16_REL + oracle.FP16_ABS * B.shape[0]
        assert np.all(np.abs(lhs - rhs) <= bound), "Freivalds (fp16) failed"
    else:
        lhs = C.astype(np.int64) @ X
        rhs = a @ (b.T @ X)
        assert np.array_equal(lhs, rhs), "Freivalds (int) failed"
