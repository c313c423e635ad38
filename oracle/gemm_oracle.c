/*
 * CPU oracle for C = A * B^T in the three precisions of the study.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code, header, table or helper
 * with the CUDA path, and nothing on the product path may call it.
 *
 * What it computes (paper Sec. II-A: a tensor-core GEMM is D = A*B + C, here
 * with C = 0; Listing 2(c): operands are ".row.col", i.e. A is M x K row-major
 * and B is stored N x K with K contiguous; Listing 1: row i of A starts at
 * A + i*K elements, K/2 bytes for 4-bit data; Sec. VI: INT32 results without
 * dequantisation or scaling):
 *
 *     C[i][j] = sum_{k=0}^{K-1} a(i,k) * b(j,k)
 *
 * Every routine is the literal triple loop i -> j -> k, k ascending, with an
 * accumulator wide enough to be exact (int64) or five orders of magnitude
 * tighter than the tolerance (fp64).  No blocking, no reordering.
 *
 * A row subset / column subset may be given (rows == NULL means all rows,
 * cols == NULL means all columns); the output is then the nr x nc block of the
 * selected rows and columns, row-major with leading dimension nc.
 *
 * Parity status: every function here is pinned (numpy int64/fp64 matmul,
 * brute force on tiny cases, closed forms, one-hot index sweeps, int32 range
 * bounds) by the CPU tests.  What stays unpinned by design is the bit pattern
 * of the GPU's FP32 accumulation: only the stated error bound is checked.
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>
#include <stdlib.h>

#define ORACLE_OK 0
#define ORACLE_BAD_ARG -1
#define ORACLE_NONFINITE -2
#define ORACLE_NO_MEMORY -3

/* IEEE binary16 -> double by bit fields.  Returns 0 and sets *ok = 0 for
 * infinities and NaNs: the GEMM inputs are finite by construction. */
static double half_bits_to_double(uint16_t h, int *ok)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int mant = h & 0x3ff;
    double v;
    if (expo == 0x1f) {
        *ok = 0;
        return 0.0;
    }
    if (expo == 0)
        v = ldexp((double)mant, -24);              /* subnormal: m * 2^-24 */
    else
        v = ldexp((double)(mant + 1024), expo - 25); /* (1 + m/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* Element k of a packed signed 4-bit row: two per byte, element 2m in the low
 * nibble of byte m, element 2m+1 in the high nibble, two's complement. */
static int nibble_at(const uint8_t *row, int k)
{
    int n = (row[k >> 1] >> (4 * (k & 1))) & 15;
    return (n ^ 8) - 8;
}

static int bad_args(int M, int N, int K, const void *A, const void *B,
                    const int32_t *rows, int nr, const int32_t *cols, int nc,
                    const void *C)
{
    int t;
    if (M <= 0 || N <= 0 || K <= 0 || !A || !B || !C || nr < 0 || nc < 0)
        return 1;
    if (rows)
        for (t = 0; t < nr; ++t)
            if (rows[t] < 0 || rows[t] >= M)
                return 1;
    if (cols)
        for (t = 0; t < nc; ++t)
            if (cols[t] < 0 || cols[t] >= N)
                return 1;
    return 0;
}

/* Step 1 of the FP16 path: decode a whole operand once.  Every binary16 value
 * is exactly representable in binary32, so the decoded copy loses nothing and
 * halves the scratch memory; products and sums are formed in fp64 below. */
static float *decode_half_matrix(const uint16_t *X, size_t count, int *ok_out)
{
    float *out = (float *)malloc(count * sizeof(float));
    int bad = 0;
    if (!out)
        return NULL;
#pragma omp parallel for schedule(static) reduction(|:bad)
    for (long long t = 0; t < (long long)count; ++t) {
        int ok = 1;
        out[t] = (float)half_bits_to_double(X[t], &ok);
        if (!ok) bad |= 1;
    }
    if (bad) *ok_out = 0;
    return out;
}

/* FP16 inputs, fp64 accumulation.  C gets the sums, S (may be NULL) gets
 * sum_k |a*b|, the quantity the FP16 error bound is stated in.  Every
 * fp16 x fp16 product has at most 22 significant bits and is exact in fp64. */
int oracle_gemm_fp16(int M, int N, int K, const uint16_t *A, const uint16_t *B,
                     const int32_t *rows, int nr, const int32_t *cols, int nc,
                     double *C, double *S)
{
    int ok = 1;
    float *a32, *b32;
    if (bad_args(M, N, K, A, B, rows, nr, cols, nc, C))
        return ORACLE_BAD_ARG;
    if (!rows) nr = M;
    if (!cols) nc = N;
    a32 = decode_half_matrix(A, (size_t)M * K, &ok);
    b32 = decode_half_matrix(B, (size_t)N * K, &ok);
    if (!a32 || !b32) {
        free(a32);
        free(b32);
        return ORACLE_NO_MEMORY;
    }
#pragma omp parallel for schedule(static)
    for (int r = 0; r < nr; ++r) {
        int i = rows ? rows[r] : r;
        for (int c = 0; c < nc; ++c) {
            int j = cols ? cols[c] : c;
            double acc = 0.0, mag = 0.0;
            for (int k = 0; k < K; ++k) {
                double p = (double)a32[(size_t)i * K + k] * (double)b32[(size_t)j * K + k];
                acc += p;
                mag += fabs(p);
            }
            C[(size_t)r * nc + c] = acc;
            if (S) S[(size_t)r * nc + c] = mag;
        }
    }
    free(a32);
    free(b32);
    return ok ? ORACLE_OK : ORACLE_NONFINITE;
}

/* Signed 8-bit inputs, exact int64 sums (the caller checks the int32 range). */
int oracle_gemm_s8(int M, int N, int K, const int8_t *A, const int8_t *B,
                   const int32_t *rows, int nr, const int32_t *cols, int nc,
                   int64_t *C)
{
    if (bad_args(M, N, K, A, B, rows, nr, cols, nc, C))
        return ORACLE_BAD_ARG;
    if (!rows) nr = M;
    if (!cols) nc = N;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < nr; ++r) {
        int i = rows ? rows[r] : r;
        for (int c = 0; c < nc; ++c) {
            int j = cols ? cols[c] : c;
            int64_t acc = 0;
            for (int k = 0; k < K; ++k)
                acc += (int64_t)A[(size_t)i * K + k] * (int64_t)B[(size_t)j * K + k];
            C[(size_t)r * nc + c] = acc;
        }
    }
    return ORACLE_OK;
}

/* Packed signed 4-bit inputs (rows of K/2 bytes; K must be even), exact
 * int64 sums. */
int oracle_gemm_s4(int M, int N, int K, const uint8_t *A, const uint8_t *B,
                   const int32_t *rows, int nr, const int32_t *cols, int nc,
                   int64_t *C)
{
    if (bad_args(M, N, K, A, B, rows, nr, cols, nc, C) || (K & 1))
        return ORACLE_BAD_ARG;
    if (!rows) nr = M;
    if (!cols) nc = N;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < nr; ++r) {
        int i = rows ? rows[r] : r;
        const uint8_t *arow = A + (size_t)i * (K / 2);
        for (int c = 0; c < nc; ++c) {
            int j = cols ? cols[c] : c;
            const uint8_t *brow = B + (size_t)j * (K / 2);
            int64_t acc = 0;
            for (int k = 0; k < K; ++k)
                acc += (int64_t)nibble_at(arow, k) * (int64_t)nibble_at(brow, k);
            C[(size_t)r * nc + c] = acc;
        }
    }
    return ORACLE_OK;
}

#ifdef _OPENMP
#include <omp.h>
int oracle_threads(void) { return omp_get_max_threads(); }
#else
int oracle_threads(void) { return 1; }
#endif
