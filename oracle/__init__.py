"""CPU oracle for the GEMM hot path.  TEST INFRASTRUCTURE ONLY.

Thin ctypes loader around ``gemm_oracle.c`` (plain C triple loops, int64 / fp64
accumulation).  Only the tests, the smoke check and the benchmark's CPU
baseline leg may import this package; the CUDA library and its Python binding
never do, and this package never imports them.

The arithmetic lives in the C file; this module only marshals numpy arrays,
narrows the exact int64 sums to int32 after a range check, and evaluates the
FP16 acceptance bound.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gemm_oracle.c")
_LIB = os.path.join(_HERE, "libgemm_oracle.so")
_lib = None

INT32_MIN = -(2 ** 31)
INT32_MAX = 2 ** 31 - 1

# Acceptance rule for the FP16 path: |C_gpu - C_ref| <= REL * sum_k|a*b| + ABS.
FP16_REL = 1e-4
FP16_ABS = 1e-6


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p = ctypes.POINTER(ctypes.c_int32)
        common = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                  ctypes.c_void_p, i32p, ctypes.c_int, i32p, ctypes.c_int]
        lib.oracle_gemm_fp16.argtypes = common + [ctypes.c_void_p, ctypes.c_void_p]
        lib.oracle_gemm_s8.argtypes = common + [ctypes.c_void_p]
        lib.oracle_gemm_s4.argtypes = common + [ctypes.c_void_p]
        for f in (lib.oracle_gemm_fp16, lib.oracle_gemm_s8, lib.oracle_gemm_s4,
                  lib.oracle_threads):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().oracle_threads())


def _index_arg(idx, limit):
    if idx is None:
        return None, 0, limit, None
    arr = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    ptr = arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    return ptr, arr.size, arr.size, arr  # keep arr alive


def _check(rc):
    if rc == -1:
        raise ValueError("oracle: bad argument (shape, index or odd K for int4)")
    if rc == -2:
        raise ValueError("oracle: non-finite fp16 input")
    if rc == -3:
        raise MemoryError("oracle: out of memory")
    if rc != 0:
        raise RuntimeError("oracle: error %d" % rc)


def gemm_fp16(A, B, rows=None, cols=None):
    """A: (M,K) float16, B: (N,K) float16.  Returns (C, S) as float64 arrays of
    shape (len(rows) or M, len(cols) or N): C = sum_k a*b, S = sum_k |a*b|."""
    A = np.ascontiguousarray(A)
    B = np.ascontiguousarray(B)
    assert A.dtype == np.float16 and B.dtype == np.float16
    assert A.ndim == 2 and B.ndim == 2 and A.shape[1] == B.shape[1]
    M, K = A.shape
    N = B.shape[0]
    rp, nr, orow, _kr = _index_arg(rows, M)
    cp, nc, ocol, _kc = _index_arg(cols, N)
    C = np.empty((orow, ocol), dtype=np.float64)
    S = np.empty((orow, ocol), dtype=np.float64)
    _check(_load().oracle_gemm_fp16(M, N, K, A.ctypes.data, B.ctypes.data,
                                    rp, nr, cp, nc, C.ctypes.data, S.ctypes.data))
    return C, S


def gemm_s8_i64(A, B, rows=None, cols=None):
    """A: (M,K) int8, B: (N,K) int8.  Exact sums as int64."""
    A = np.ascontiguousarray(A)
    B = np.ascontiguousarray(B)
    assert A.dtype == np.int8 and B.dtype == np.int8
    assert A.ndim == 2 and B.ndim == 2 and A.shape[1] == B.shape[1]
    M, K = A.shape
    N = B.shape[0]
    rp, nr, orow, _kr = _index_arg(rows, M)
    cp, nc, ocol, _kc = _index_arg(cols, N)
    C = np.empty((orow, ocol), dtype=np.int64)
    _check(_load().oracle_gemm_s8(M, N, K, A.ctypes.data, B.ctypes.data,
                                  rp, nr, cp, nc, C.ctypes.data))
    return C


def gemm_s4_i64(A, B, K, rows=None, cols=None):
    """A: (M,K/2) uint8, B: (N,K/2) uint8, packed two signed 4-bit values per
    byte, low nibble first.  Exact sums as int64."""
    A = np.ascontiguousarray(A)
    B = np.ascontiguousarray(B)
    assert A.dtype == np.uint8 and B.dtype == np.uint8
    assert A.ndim == 2 and B.ndim == 2
    assert K % 2 == 0 and A.shape[1] == K // 2 and B.shape[1] == K // 2
    M = A.shape[0]
    N = B.shape[0]
    rp, nr, orow, _kr = _index_arg(rows, M)
    cp, nc, ocol, _kc = _index_arg(cols, N)
    C = np.empty((orow, ocol), dtype=np.int64)
    _check(_load().oracle_gemm_s4(M, N, K, A.ctypes.data, B.ctypes.data,
                                  rp, nr, cp, nc, C.ctypes.data))
    return C


def narrow_int32(C64):
    """Range check, then narrow: the INT32 result is only defined when every
    exact sum fits (the paper's accumulators are s32; overflow is out of
    domain)."""
    if C64.size and (C64.min() < INT32_MIN or C64.max() > INT32_MAX):
        raise OverflowError("oracle: exact sum outside the int32 range")
    return C64.astype(np.int32)


def gemm_s8(A, B, rows=None, cols=None):
    return narrow_int32(gemm_s8_i64(A, B, rows, cols))


def gemm_s4(A, B, K, rows=None, cols=None):
    return narrow_int32(gemm_s4_i64(A, B, K, rows, cols))


def fp16_bound(S):
    """Per-element acceptance bound for the FP16 path, in fp64."""
    return FP16_REL * np.asarray(S, dtype=np.float64) + FP16_ABS


def fp16_check(C_got, C_ref, S):
    """Returns (ok, worst): every element finite and inside the bound;
    worst = max |err| / bound."""
    got = np.asarray(C_got, dtype=np.float64)
    if got.shape != C_ref.shape:
        return False, float("inf")
    if got.size == 0:
        return True, 0.0
    if not np.isfinite(got).all():
        return False, float("inf")
    ratio = np.abs(got - C_ref) / fp16_bound(S)
    worst = float(ratio.max())
    return worst <= 1.0, worst


# ---------------------------------------------------------------------------
# Output variants: FP16-rounded C and dequantised integer GEMM.  The reference
# values are the exact sums above pushed through the definition in fp64; the
# bounds add the roundings the definition allows.
# ---------------------------------------------------------------------------
HALF_EPS = 2.0 ** -11          # half an ulp of binary16, relative (normal range)
HALF_TINY = 2.0 ** -25         # half the smallest binary16 subnormal
FLOAT_EPS = 2.0 ** -24         # half an ulp of binary32, relative


def fp16_out_bound(C_ref, S):
    """FP32-accumulate bound plus one rounding of the result to binary16."""
    return fp16_bound(S) + HALF_EPS * np.abs(C_ref) + HALF_TINY


def fp16_out_check(C_got, C_ref, S):
    got = np.asarray(C_got)
    if got.dtype != np.float16 or got.shape != C_ref.shape:
        return False, float("inf")
    got = got.astype(np.float64)
    if got.size == 0:
        return True, 0.0
    if not np.isfinite(got).all():
        return False, float("inf")
    ratio = np.abs(got - C_ref) / fp16_out_bound(C_ref, S)
    worst = float(ratio.max())
    return worst <= 1.0, worst


def dequant_ref(C64, row_scale, col_scale):
    """C[i][j] = sum * row_scale[i] * col_scale[j], in fp64 from the exact integer sums."""
    rs = np.asarray(row_scale, dtype=np.float32).astype(np.float64)
    cs = np.asarray(col_scale, dtype=np.float32).astype(np.float64)
    assert C64.shape == (rs.size, cs.size)
    return C64.astype(np.float64) * rs[:, None] * cs[None, :]


def dequant_check(C_got, ref, out_is_fp16):
    """The definition allows three FP32 roundings (int -> float, two products) and, for
    binary16 output, one more; the bound is their sum with a 2x margin on the FP32 part."""
    got = np.asarray(C_got)
    want_dtype = np.float16 if out_is_fp16 else np.float32
    if got.dtype != want_dtype or got.shape != ref.shape:
        return False, float("inf")
    got = got.astype(np.float64)
    if got.size == 0:
        return True, 0.0
    if not np.isfinite(got).all():
        return False, float("inf")
    bound = 6 * FLOAT_EPS * np.abs(ref) + 1e-37
    if out_is_fp16:
        bound = bound + HALF_EPS * np.abs(ref) + HALF_TINY
    ratio = np.abs(got - ref) / bound
    worst = float(ratio.max())
    return worst <= 1.0, worst
