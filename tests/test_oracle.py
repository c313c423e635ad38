"""Pins for the CPU oracle: every check here compares the oracle with
something that is not the oracle (a library matmul on separately decoded
inputs, Python big-integer / Fraction brute force, closed forms, hand-written
expected values)."""
from fractions import Fraction

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2608_10103_b200 import synth


def unpack_s4_py(P, K):
    """Independent nibble decoder (numpy, not the oracle's)."""
    lo = (P & 0x0F).astype(np.int16)
    hi = (P >> 4).astype(np.int16)
    out = np.empty((P.shape[0], K), dtype=np.int16)
    out[:, 0::2] = np.where(lo >= 8, lo - 16, lo)
    out[:, 1::2] = np.where(hi >= 8, hi - 16, hi)
    return out


# ----------------------------------------------------------------- library pins
@pytest.mark.parametrize("M,N,K", [(64, 48, 96), (130, 257, 320), (300, 200, 512)])
def test_s8_matches_numpy_int64(M, N, K):
    A, B = synth.s8_uniform(M, N, K, seed=101)
    want = A.astype(np.int64) @ B.astype(np.int64).T
    assert np.array_equal(oracle.gemm_s8_i64(A, B), want)
    assert np.array_equal(oracle.gemm_s8(A, B), want.astype(np.int32))


@pytest.mark.parametrize("M,N,K", [(64, 48, 96), (130, 257, 320), (300, 200, 512)])
def test_s4_matches_numpy_int64(M, N, K):
    A, B = synth.s4_uniform(M, N, K, seed=102)
    a = unpack_s4_py(A, K).astype(np.int64)
    b = unpack_s4_py(B, K).astype(np.int64)
    assert np.array_equal(oracle.gemm_s4_i64(A, B, K), a @ b.T)


def test_s4_equals_s8_on_unpacked():
    M, N, K = 70, 90, 128
    A, B = synth.s4_uniform(M, N, K, seed=103)
    a8 = unpack_s4_py(A, K).astype(np.int8)
    b8 = unpack_s4_py(B, K).astype(np.int8)
    assert np.array_equal(oracle.gemm_s4_i64(A, B, K), oracle.gemm_s8_i64(a8, b8))


@pytest.mark.parametrize("gen", [synth.fp16_uniform, synth.fp16_normal_clipped])
def test_fp16_matches_dgemm(gen):
    M, N, K = 150, 170, 384
    A, B = gen(M, N, K, seed=104)
    C, S = oracle.gemm_fp16(A, B)
    a = A.astype(np.float64)
    b = B.astype(np.float64)
    want = a @ b.T
    wantS = np.abs(a) @ np.abs(b).T
    assert np.all(np.abs(C - want) <= 1e-12 * wantS + 1e-300)
    assert np.all(np.abs(S - wantS) <= 1e-12 * wantS + 1e-300)


def test_fp16_decoder_all_finite_patterns():
    """C[i][0] = value(bits i) * 1: pins the bit-field decoder (normals,
    subnormals, both zeros) against numpy's own half -> double conversion."""
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    h = bits.view(np.float16)
    finite = np.isfinite(h)
    A = np.zeros((int(finite.sum()), 2), dtype=np.float16)
    A[:, 0] = h[finite]
    B = np.array([[1.0, 0.0]], dtype=np.float16)
    C, S = oracle.gemm_fp16(A, B)
    want = h[finite].astype(np.float64)
    assert np.array_equal(C[:, 0], want)
    assert np.array_equal(S[:, 0], np.abs(want))


@pytest.mark.parametrize("bad", [0x7C00, 0xFC00, 0x7E00, 0x7C01])
def test_fp16_rejects_nonfinite(bad):
    A = np.array([[bad, 0]], dtype=np.uint16).view(np.float16)
    B = np.ones((1, 2), dtype=np.float16)
    with pytest.raises(ValueError):
        oracle.gemm_fp16(A, B)


# -------------------------------------------------------- hand-written tiny cases
def test_tiny_s8_by_hand():
    A = np.array([[1, -2, 3, 4], [-128, 127, 0, 5]], dtype=np.int8)
    B = np.array([[2, 0, -1, 1], [-128, -128, 7, -3]], dtype=np.int8)
    # row0.row0 = 2+0-3+4 = 3 ; row0.row1 = -128+256+21-12 = 137
    # row1.row0 = -256+0+0+5 = -251 ; row1.row1 = 16384-16256+0-15 = 113
    assert oracle.gemm_s8(A, B).tolist() == [[3, 137], [-251, 113]]


def test_tiny_s4_by_hand_bytes():
    # bytes written out by hand: low nibble = even k, high nibble = odd k
    # A row0 = [1, -1, 7, -8] -> 0xF1, 0x87 ; row1 = [0, 2, -3, 4] -> 0x20, 0x4D
    # B row0 = [-8, -8, 7, 7] -> 0x88, 0x77 ; row1 = [3, 0, 0, -1] -> 0x03, 0xF0
    A = np.array([[0xF1, 0x87], [0x20, 0x4D]], dtype=np.uint8)
    B = np.array([[0x88, 0x77], [0x03, 0xF0]], dtype=np.uint8)
    # r0.b0 = -8+8+49-56 = -7 ; r0.b1 = 3+0+0+8 = 11
    # r1.b0 = 0-16-21+28 = -9 ; r1.b1 = 0+0+0-4 = -4
    assert oracle.gemm_s4(A, B, 4).tolist() == [[-7, 11], [-9, -4]]


def test_tiny_fp16_by_hand():
    A = np.array([[1.5, -2.0, 0.25, 0.0]], dtype=np.float16)
    B = np.array([[2.0, 0.5, -4.0, 9.0], [6.1035e-05, 1.0, 1.0, 1.0]], dtype=np.float16)
    C, S = oracle.gemm_fp16(A, B)
    assert C[0, 0] == 3.0 - 1.0 - 1.0
    assert S[0, 0] == 5.0
    assert C[0, 1] == 1.5 * 2.0 ** -14 - 2.0 + 0.25


# ------------------------------------------------------------ brute force (exact)
@settings(max_examples=40, deadline=None)
@given(st.integers(1, 5), st.integers(1, 5), st.integers(1, 9), st.integers(0, 2 ** 31))
def test_s8_brute_force(M, N, K, seed):
    A, B = synth.s8_uniform(M, N, K, seed)
    got = oracle.gemm_s8_i64(A, B)
    for i in range(M):
        for j in range(N):
            assert int(got[i, j]) == sum(int(A[i, k]) * int(B[j, k]) for k in range(K))


@settings(max_examples=40, deadline=None)
@given(st.integers(1, 5), st.integers(1, 5), st.integers(1, 6), st.integers(0, 2 ** 31))
def test_s4_brute_force(M, N, K2, seed):
    K = 2 * K2
    g = np.random.Generator(np.random.PCG64(seed))
    a = g.integers(-8, 8, size=(M, K))
    b = g.integers(-8, 8, size=(N, K))
    got = oracle.gemm_s4_i64(synth.pack_s4(a), synth.pack_s4(b), K)
    for i in range(M):
        for j in range(N):
            assert int(got[i, j]) == sum(int(a[i, k]) * int(b[j, k]) for k in range(K))


@settings(max_examples=25, deadline=None)
@given(st.integers(1, 4), st.integers(1, 4), st.integers(1, 8), st.integers(0, 2 ** 31))
def test_fp16_brute_force_fraction(M, N, K, seed):
    A, B = synth.fp16_normal_clipped(M, N, K, seed)
    C, S = oracle.gemm_fp16(A, B)
    for i in range(M):
        for j in range(N):
            exact = sum(Fraction(float(A[i, k])) * Fraction(float(B[j, k])) for k in range(K))
            mag = sum(abs(Fraction(float(A[i, k])) * Fraction(float(B[j, k]))) for k in range(K))
            assert abs(Fraction(float(C[i, j])) - exact) <= mag * Fraction(K, 2 ** 52)
            assert abs(Fraction(float(S[i, j])) - mag) <= mag * Fraction(K, 2 ** 52)


# ------------------------------------------------------------------- closed forms
@pytest.mark.parametrize("K", [2, 64, 512, 4096])
def test_all_ones_gives_K(K):
    M, N = 5, 7
    assert np.all(oracle.gemm_s8_i64(np.ones((M, K), np.int8), np.ones((N, K), np.int8)) == K)
    ones4 = synth.pack_s4(np.ones((max(M, N), K), np.int8))
    assert np.all(oracle.gemm_s4_i64(ones4[:M], ones4[:N], K) == K)
    C, S = oracle.gemm_fp16(np.ones((M, K), np.float16), np.ones((N, K), np.float16))
    assert np.all(C == K) and np.all(S == K)


def test_identity_operands():
    K = 96
    eye = np.eye(K, dtype=np.int8)
    A, B = synth.s8_uniform(40, 56, K, seed=7)
    assert np.array_equal(oracle.gemm_s8_i64(A, eye), A.astype(np.int64))      # B = I -> C = A
    assert np.array_equal(oracle.gemm_s8_i64(eye, B), B.T.astype(np.int64))    # A = I -> C = B^T
    g = np.random.Generator(np.random.PCG64(8))
    a = g.integers(-8, 8, size=(40, K))
    assert np.array_equal(oracle.gemm_s4_i64(synth.pack_s4(a), synth.pack_s4(eye), K), a)
    assert np.array_equal(oracle.gemm_s4_i64(synth.pack_s4(eye), synth.pack_s4(a), K), a.T)
    Af, Bf = synth.fp16_uniform(40, 56, K, seed=9)
    C, _ = oracle.gemm_fp16(Af, np.eye(K, dtype=np.float16))
    assert np.array_equal(C, Af.astype(np.float64))
    C, _ = oracle.gemm_fp16(np.eye(K, dtype=np.float16), Bf)
    assert np.array_equal(C, Bf.T.astype(np.float64))


def test_rank_one_and_alternating():
    M, N, K = 9, 11, 64
    x = np.arange(M) - 4
    y = np.arange(N) - 5
    A = np.repeat(x[:, None], K, axis=1)
    B = np.repeat(y[:, None], K, axis=1)
    want = K * np.outer(x, y)
    assert np.array_equal(oracle.gemm_s8_i64(A.astype(np.int8), B.astype(np.int8)), want)
    assert np.array_equal(oracle.gemm_s4_i64(synth.pack_s4(A), synth.pack_s4(B), K), want)
    C, _ = oracle.gemm_fp16(A.astype(np.float16), B.astype(np.float16))
    assert np.array_equal(C, want.astype(np.float64))
    sign = np.where(np.arange(K) % 2 == 0, 1, -1)
    Aalt = (A * sign).astype(np.int8)
    assert np.all(oracle.gemm_s8_i64(Aalt, B.astype(np.int8)) == 0)
    assert np.all(oracle.gemm_s4_i64(synth.pack_s4(A * sign), synth.pack_s4(B), K) == 0)


# ------------------------------------------------------------- int32 range bounds
def test_int32_range_bounds():
    K = 8192
    lo8 = np.full((2, K), -128, np.int8)
    hi8 = np.full((2, K), 127, np.int8)
    assert np.all(oracle.gemm_s8_i64(lo8, lo8) == 16384 * K) and 16384 * K == 2 ** 27
    assert np.all(oracle.gemm_s8_i64(lo8, hi8) == -16256 * K) and -16256 * K == -133169152
    assert np.all(oracle.gemm_s8(lo8, lo8) == 2 ** 27)
    lo4 = synth.pack_s4(np.full((2, K), -8))
    hi4 = synth.pack_s4(np.full((2, K), 7))
    assert np.all(oracle.gemm_s4_i64(lo4, lo4, K) == 524288)
    assert np.all(oracle.gemm_s4_i64(lo4, hi4, K) == -458752)


def test_narrowing_rejects_overflow():
    # the largest K whose worst case still fits is 131071: 16384*131072 = 2^31 overflows
    assert 16384 * 131071 <= oracle.INT32_MAX < 16384 * 131072
    with pytest.raises(OverflowError):
        oracle.narrow_int32(np.array([[2 ** 31]], dtype=np.int64))
    with pytest.raises(OverflowError):
        oracle.narrow_int32(np.array([[-2 ** 31 - 1]], dtype=np.int64))
    assert oracle.narrow_int32(np.array([[2 ** 31 - 1, -2 ** 31]], dtype=np.int64)).tolist() == [
        [2 ** 31 - 1, -2 ** 31]]
    K = 131072
    lo8 = np.full((1, K), -128, np.int8)
    assert oracle.gemm_s8_i64(lo8, lo8)[0, 0] == 2 ** 31
    with pytest.raises(OverflowError):
        oracle.gemm_s8(lo8, lo8)


# ------------------------------------------------- nibble order and sign extension
def test_s4_one_hot_positions():
    K = 256
    ks = [0, 1, 2, 31, 32, 63, 64, 127, 128, K - 1]
    a = np.zeros((len(ks), K), dtype=np.int8)
    b = np.zeros((len(ks), K), dtype=np.int8)
    for r, k in enumerate(ks):
        a[r, k] = 1
        b[r, k] = 1
    got = oracle.gemm_s4_i64(synth.pack_s4(a), synth.pack_s4(b), K)
    assert np.array_equal(got, np.eye(len(ks), dtype=np.int64))
    # the same through hand-made bytes: element k lives in byte k>>1, nibble k&1
    A = np.zeros((len(ks), K // 2), dtype=np.uint8)
    for r, k in enumerate(ks):
        A[r, k >> 1] = 1 << (4 * (k & 1))
    assert np.array_equal(oracle.gemm_s4_i64(A, A, K), np.eye(len(ks), dtype=np.int64))


def test_s4_even_odd_never_meet():
    K = 64
    A = np.full((3, K // 2), 0x07, dtype=np.uint8)   # 7 on even k, 0 on odd k
    B = np.full((4, K // 2), 0x90, dtype=np.uint8)   # 0 on even k, -7 on odd k
    assert np.all(oracle.gemm_s4_i64(A, B, K) == 0)
    assert np.all(oracle.gemm_s4_i64(A, A, K) == 49 * (K // 2))
    assert np.all(oracle.gemm_s4_i64(B, B, K) == 49 * (K // 2))


def test_s4_value_sweep():
    K = 32
    ones = np.full((1, K // 2), 0x11, dtype=np.uint8)
    for v in range(-8, 8):
        n = v & 15
        A = np.full((1, K // 2), n | (n << 4), dtype=np.uint8)
        assert oracle.gemm_s4_i64(A, ones, K)[0, 0] == K * v


def test_s8_value_sweep():
    K = 16
    ones = np.ones((1, K), dtype=np.int8)
    for v in range(-128, 128):
        assert oracle.gemm_s8_i64(np.full((1, K), v, np.int8), ones)[0, 0] == K * v


# ------------------------------------------------------------------ index mapping
def test_row_and_column_indexing():
    M, N, K = 300, 270, 32
    a = np.zeros((M, K), np.int8)
    b = np.zeros((N, K), np.int8)
    a[:, 0] = (np.arange(M) % 97) - 48
    b[:, 0] = (np.arange(N) % 89) - 44
    want = np.outer(a[:, 0].astype(np.int64), b[:, 0].astype(np.int64))
    assert np.array_equal(oracle.gemm_s8_i64(a, b), want)
    a4 = np.clip(a, -8, 7)
    b4 = np.clip(b, -8, 7)
    want4 = np.outer(a4[:, 0].astype(np.int64), b4[:, 0].astype(np.int64))
    assert np.array_equal(oracle.gemm_s4_i64(synth.pack_s4(a4), synth.pack_s4(b4), K), want4)


def test_subset_mode_matches_full():
    M, N, K = 90, 75, 64
    rows = np.array([0, 89, 17, 17, 42], dtype=np.int32)
    cols = np.array([74, 0, 33], dtype=np.int32)
    A, B = synth.s8_uniform(M, N, K, seed=21)
    full = A.astype(np.int64) @ B.astype(np.int64).T
    assert np.array_equal(oracle.gemm_s8_i64(A, B, rows=rows), full[rows])
    assert np.array_equal(oracle.gemm_s8_i64(A, B, cols=cols), full[:, cols])
    assert np.array_equal(oracle.gemm_s8_i64(A, B, rows, cols), full[np.ix_(rows, cols)])
    A4, B4 = synth.s4_uniform(M, N, K, seed=22)
    full4 = unpack_s4_py(A4, K).astype(np.int64) @ unpack_s4_py(B4, K).astype(np.int64).T
    assert np.array_equal(oracle.gemm_s4_i64(A4, B4, K, rows, cols), full4[np.ix_(rows, cols)])
    Af, Bf = synth.fp16_uniform(M, N, K, seed=23)
    fullf = Af.astype(np.float64) @ Bf.astype(np.float64).T
    C, S = oracle.gemm_fp16(Af, Bf, rows, cols)
    assert np.allclose(C, fullf[np.ix_(rows, cols)], rtol=0, atol=1e-12 * K)
    with pytest.raises(ValueError):
        oracle.gemm_s8_i64(A, B, rows=np.array([M], dtype=np.int32))
    with pytest.raises(ValueError):
        oracle.gemm_s8_i64(A, B, cols=np.array([-1], dtype=np.int32))


# --------------------------------------------------------------------- invariants
def test_invariants_int():
    M, N, K = 33, 47, 160
    A, B = synth.s8_uniform(M, N, K, seed=31)
    C = oracle.gemm_s8_i64(A, B)
    assert np.array_equal(oracle.gemm_s8_i64(B, A), C.T)                       # transpose symmetry
    perm = np.random.Generator(np.random.PCG64(5)).permutation(K)
    assert np.array_equal(oracle.gemm_s8_i64(A[:, perm], B[:, perm]), C)        # K-permutation
    C1 = oracle.gemm_s8_i64(np.ascontiguousarray(A[:, :64]), np.ascontiguousarray(B[:, :64]))
    C2 = oracle.gemm_s8_i64(np.ascontiguousarray(A[:, 64:]), np.ascontiguousarray(B[:, 64:]))
    assert np.array_equal(C1 + C2, C)                                           # additivity over K
    A2 = (A // 2).astype(np.int8)
    A3 = (A - A2).astype(np.int8)
    assert np.array_equal(oracle.gemm_s8_i64(A2, B) + oracle.gemm_s8_i64(A3, B), C)  # linearity


def test_invariants_fp16():
    M, N, K = 20, 30, 128
    A, B = synth.fp16_uniform(M, N, K, seed=32)
    C, S = oracle.gemm_fp16(A, B)
    Ct, St = oracle.gemm_fp16(B, A)
    assert np.array_equal(Ct, C.T) and np.array_equal(St, S.T)
    perm = np.random.Generator(np.random.PCG64(6)).permutation(K)
    Cp, _ = oracle.gemm_fp16(A[:, perm], B[:, perm])
    assert np.all(np.abs(Cp - C) <= 1e-12 * S)
    assert np.all(S >= np.abs(C))


# ------------------------------------------------------ tolerance rule and metric
def test_fp16_check_rule():
    Cref = np.array([[1.0, -2.0]])
    S = np.array([[10.0, 0.0]])
    assert oracle.fp16_check(np.array([[1.0 + 1.0e-3, -2.0 + 1e-6]]), Cref, S)[0]
    assert not oracle.fp16_check(np.array([[1.0 + 1.1e-3, -2.0]]), Cref, S)[0]
    assert not oracle.fp16_check(np.array([[1.0, -2.0 + 1.1e-6]]), Cref, S)[0]
    assert not oracle.fp16_check(np.array([[np.nan, -2.0]]), Cref, S)[0]
    assert not oracle.fp16_check(np.array([[1.0]]), Cref, S)[0]


def test_fp32_sequential_accumulation_is_far_inside_bound():
    """The bound leaves room for any FP32 accumulation order: a plain fp32
    running sum over K = 1024 lands two orders of magnitude inside it."""
    M, N, K = 16, 16, 1024
    A, B = synth.fp16_uniform(M, N, K, seed=33)
    C, S = oracle.gemm_fp16(A, B)
    acc = np.zeros((M, N), dtype=np.float32)
    a32 = A.astype(np.float32)
    b32 = B.astype(np.float32)
    for k in range(K):
        acc = (acc + np.outer(a32[:, k], b32[:, k]).astype(np.float32)).astype(np.float32)
    ok, worst = oracle.fp16_check(acc, C, S)
    assert ok and worst < 0.05


def test_ops_convention_matches_paper_table(golden_dir):
    rows = [l.split() for l in open(golden_dir + "/table2_tops_n8192.txt")
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for name, n, ms, tops in rows:
        n = int(n)
        derived = synth.gemm_ops(n, n, n) / (float(ms) * 1e-3) / 1e12
        assert abs(derived - float(tops)) <= 0.012 * float(tops) + 5e-4, name


# ------------------------------------------------------- output-variant references
def test_fp16_out_bound_by_hand():
    ref = np.array([[1.0 + 2.0 ** -11, 1000.0, 2.0 ** -26]])
    S = np.zeros_like(ref)
    # nearest halfs: 1.0 (tie -> even) or 1+2^-10, 1000.0, 0.0 -- all inside the bound
    assert oracle.fp16_out_check(np.array([[1.0, 1000.0, 0.0]], np.float16), ref, S)[0]
    assert oracle.fp16_out_check(np.array([[1.0 + 2.0 ** -10, 1000.0, 0.0]], np.float16), ref, S)[0]
    # one half-ulp further is outside: 1 + 2^-9, 1001
    assert not oracle.fp16_out_check(np.array([[1.0 + 2.0 ** -9, 1000.0, 0.0]], np.float16), ref, S)[0]
    assert not oracle.fp16_out_check(np.array([[1.0, 1001.0, 0.0]], np.float16), ref, S)[0]
    assert not oracle.fp16_out_check(np.array([[1.0, 1000.0, 0.0]], np.float32), ref, S)[0]


def test_dequant_reference_by_hand():
    C = np.array([[4, -6], [10, 0]], dtype=np.int64)
    ref = oracle.dequant_ref(C, np.array([0.5, 2.0], np.float32), np.array([3.0, -0.25], np.float32))
    assert ref.tolist() == [[6.0, 0.75], [60.0, -0.0]]
    assert oracle.dequant_check(ref.astype(np.float32), ref, False)[0]
    assert oracle.dequant_check(ref.astype(np.float16), ref, True)[0]
    bad = ref.astype(np.float32)
    bad[0, 0] = np.nextafter(np.float32(6.0), np.float32(7.0), dtype=np.float32) * np.float32(1 + 1e-5)
    assert not oracle.dequant_check(bad, ref, False)[0]
    assert not oracle.dequant_check(ref.astype(np.float32), ref, True)[0]
    # scales are taken at float32 precision: 0.1 means float32(0.1)
    r = oracle.dequant_ref(np.array([[10]], np.int64), [0.1], [1.0])
    assert r[0, 0] == 10 * float(np.float32(0.1))
