/*
 * oracle_gemm.c -- CPU oracle for dense GEMM.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked
 * against.  It is used by the tests, by the smoke check and by the timed
 * "cpu baseline" leg of the benchmark, and by nothing else: the product path
 * never calls it and shares no code, header, table or helper with it.
 *
 * What it computes (paper section 2.2, "Matrix Multiplication": A is m x k,
 * B is k x n, C = A x B is m x n, every matrix row-major, elements stored as
 * fp32 or fp16; each C[i][j] is the dot product of row i of A with column j
 * of B).  The library's boundary widens that statement to the usual BLAS
 * form, restated for row-major storage:
 *
 *     acc(i,j) = sum_{k=0}^{K-1} opA(i,k) * opB(k,j)          (fp64, k ascending)
 *     S(i,j)   = sum_{k=0}^{K-1} |opA(i,k)| * |opB(k,j)|      (for error bounds)
 *     ref(i,j) = alpha*acc(i,j) + (beta == 0 ? 0 : beta*C0(i,j))   (left in fp64)
 *
 *     opA(i,k) = transA ? A[k*lda + i] : A[i*lda + k]
 *     opB(k,j) = transB ? B[j*ldb + k] : B[k*ldb + j]
 *     C0(i,j)  = C0[i*ldc + j]
 *
 * oracle_bias_act() applies the fused tail, ref + bias[j] followed by ReLU or GELU, on top of that, and
 * oracle_residual_add() the residual matrix that may follow the activation.
 *
 * Stored elements (binary16, bfloat16, binary32) are decoded to double by the
 * bit-level decoders below, exactly; nothing here includes a CUDA header.
 * bfloat16, alpha, beta, op() and leading dimensions are not in the paper;
 * they follow the reference-BLAS meaning of GEMM.
 *
 * Pins (tests/test_oracle_*.py): the decoders against every 16-bit pattern;
 * the sum against identity / permutation matrices, rank-1 closed forms, exact
 * small-integer cases, alpha/beta invariants and numpy's float64 matmul; the
 * rounding routine against IEEE conversions done by numpy.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F16 = 0, ORACLE_BF16 = 1, ORACLE_F32 = 2, ORACLE_E4M3 = 3, ORACLE_E5M2 = 4 };

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_NO_MEM = 2 };

/* ---- decoders: stored bits -> exact double ------------------------------ */

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
double oracle_decode_f16(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24); /* subnormal: f * 2^-10 * 2^-14 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(1024 + f), e - 25); /* (1 + f/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* bfloat16: 1 sign, 8 exponent (bias 127), 7 fraction bits. */
double oracle_decode_bf16(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int f = h & 0x7f;
    double v;
    if (e == 0)
        v = ldexp((double)f, -133); /* f * 2^-7 * 2^-126 */
    else if (e == 255)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(128 + f), e - 134); /* (1 + f/128) * 2^(e-127) */
    return sign ? -v : v;
}

/* IEEE binary32: 1 sign, 8 exponent (bias 127), 23 fraction bits. */
double oracle_decode_f32(uint32_t w)
{
    int sign = (int)(w >> 31);
    int e = (int)((w >> 23) & 0xff);
    int64_t f = (int64_t)(w & 0x7fffff);
    double v;
    if (e == 0)
        v = ldexp((double)f, -149);
    else if (e == 255)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(8388608 + f), e - 150);
    return sign ? -v : v;
}

/* 8-bit float E4M3 ("fn" flavour used by GPUs; the paper only mentions fp8 as an existing type, section 2.1):
 * 1 sign, 4 exponent (bias 7), 3 fraction bits; no infinities; only S.1111.111 is NaN; largest value 448. */
double oracle_decode_e4m3(uint8_t b)
{
    int sign = (b >> 7) & 1;
    int e = (b >> 3) & 0xf;
    int f = b & 7;
    double v;
    if (e == 15 && f == 7)
        v = NAN;
    else if (e == 0)
        v = ldexp((double)f, -9); /* subnormal: f * 2^-3 * 2^-6 */
    else
        v = ldexp((double)(8 + f), e - 10); /* (1 + f/8) * 2^(e-7) */
    return sign ? -v : v;
}

/* 8-bit float E5M2: 1 sign, 5 exponent (bias 15), 2 fraction bits; IEEE-style infinities and NaNs. */
double oracle_decode_e5m2(uint8_t b)
{
    int sign = (b >> 7) & 1;
    int e = (b >> 2) & 0x1f;
    int f = b & 3;
    double v;
    if (e == 0)
        v = ldexp((double)f, -16); /* f * 2^-2 * 2^-14 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(4 + f), e - 17); /* (1 + f/4) * 2^(e-15) */
    return sign ? -v : v;
}

static size_t elem_size(int t)
{
    return t == ORACLE_F32 ? 4 : (t == ORACLE_E4M3 || t == ORACLE_E5M2) ? 1 : 2;
}

static double load_elem(int t, const void *base, int64_t idx)
{
    if (t == ORACLE_F16)
        return oracle_decode_f16(((const uint16_t *)base)[idx]);
    if (t == ORACLE_BF16)
        return oracle_decode_bf16(((const uint16_t *)base)[idx]);
    if (t == ORACLE_E4M3)
        return oracle_decode_e4m3(((const uint8_t *)base)[idx]);
    if (t == ORACLE_E5M2)
        return oracle_decode_e5m2(((const uint8_t *)base)[idx]);
    return oracle_decode_f32(((const uint32_t *)base)[idx]);
}

/* ---- rounding: double -> stored bits, one rounding, ties to even -------- */

/* Round x to a binary format with `p` significand bits (hidden bit included),
 * minimum normal exponent `emin` and maximum exponent `emax`; returns the
 * rounded value as a double (+-inf on overflow).  The quantum at x is
 * 2^(max(floor(log2|x|), emin) - (p-1)); x/quantum is exact in double, rint()
 * rounds it to nearest-even in the default rounding mode. */
static double round_to_format(double x, int p, int emin, int emax)
{
    if (isnan(x) || isinf(x) || x == 0.0)
        return x;
    int ex;
    (void)frexp(x, &ex); /* |x| = m * 2^ex, m in [0.5,1)  ->  floor(log2|x|) = ex-1 */
    int e = ex - 1;
    if (e < emin)
        e = emin;
    int q = e - (p - 1);
    double r = ldexp(rint(ldexp(x, -q)), q);
    if (fabs(r) >= ldexp(1.0, emax + 1))
        return x < 0 ? -INFINITY : INFINITY;
    return r;
}

static uint32_t encode_bits(double r, int p, int emin, int ebits)
{
    /* r is exactly representable in the target format (or inf / nan / 0). */
    uint32_t sign = signbit(r) ? 1u : 0u;
    int fbits = p - 1;
    uint32_t emask = (1u << ebits) - 1u;
    uint32_t out;
    if (isnan(r))
        out = (emask << fbits) | (1u << (fbits - 1));
    else if (isinf(r))
        out = emask << fbits;
    else if (r == 0.0)
        out = 0;
    else {
        int ex;
        double a = fabs(r);
        (void)frexp(a, &ex);
        int e = ex - 1;
        if (e < emin) {
            /* subnormal: value = f * 2^(emin - fbits) */
            out = (uint32_t)ldexp(a, -(emin - fbits));
        } else {
            uint32_t sig = (uint32_t)ldexp(a, fbits - e); /* 2^fbits + f */
            out = ((uint32_t)(e - emin + 1) << fbits) | (sig - (1u << fbits));
        }
    }
    return out | (sign << (ebits + fbits));
}

/* Round n doubles to `type` and write the stored bit patterns to `out`
 * (uint16 for F16 / BF16, uint32 for F32). */
int oracle_round(int type, const double *x, int64_t n, void *out)
{
    if (n < 0 || (n > 0 && (!x || !out)))
        return ORACLE_BAD_ARG;
    for (int64_t t = 0; t < n; ++t) {
        if (type == ORACLE_F16)
            ((uint16_t *)out)[t] = (uint16_t)encode_bits(round_to_format(x[t], 11, -14, 15), 11, -14, 5);
        else if (type == ORACLE_BF16)
            ((uint16_t *)out)[t] = (uint16_t)encode_bits(round_to_format(x[t], 8, -126, 127), 8, -126, 8);
        else if (type == ORACLE_F32)
            ((uint32_t *)out)[t] = encode_bits(round_to_format(x[t], 24, -126, 127), 24, -126, 8);
        else
            return ORACLE_BAD_ARG;
    }
    return ORACLE_OK;
}

/* ---- argument checks ----------------------------------------------------- */

static int check_args(int in_type, int c_type, int transA, int transB, int64_t M, int64_t N, int64_t K,
                      int64_t lda, int64_t ldb, int64_t ldc)
{
    if (in_type < 0 || in_type > 4 || c_type < 0 || c_type > 2)
        return ORACLE_BAD_ARG;
    if ((transA != 0 && transA != 1) || (transB != 0 && transB != 1))
        return ORACLE_BAD_ARG;
    if (M < 0 || N < 0 || K < 0)
        return ORACLE_BAD_ARG;
    if (lda < (transA ? M : K) || ldb < (transB ? K : N) || ldc < N)
        return ORACLE_BAD_ARG;
    return ORACLE_OK;
}

/* ---- the definition, one output element at a time ----------------------- */

/* ref / S for the listed (si[t], sj[t]) pairs; S may be NULL.  This is the
 * definition written out literally: one k-ascending loop per element. */
int oracle_gemm_points(int in_type, int c_type, int transA, int transB, int64_t M, int64_t N, int64_t K,
                       double alpha, const void *A, int64_t lda, const void *B, int64_t ldb, double beta,
                       const void *C0, int64_t ldc, int64_t ns, const int64_t *si, const int64_t *sj,
                       double *ref, double *S)
{
    int rc = check_args(in_type, c_type, transA, transB, M, N, K, lda, ldb, ldc);
    if (rc)
        return rc;
    if (ns < 0 || (ns > 0 && (!si || !sj || !ref)))
        return ORACLE_BAD_ARG;
    if (beta != 0.0 && !C0 && ns > 0)
        return ORACLE_BAD_ARG;
    for (int64_t t = 0; t < ns; ++t)
        if (si[t] < 0 || si[t] >= M || sj[t] < 0 || sj[t] >= N)
            return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < ns; ++t) {
        int64_t i = si[t], j = sj[t];
        double acc = 0.0, s = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = load_elem(in_type, A, transA ? k * lda + i : i * lda + k);
            double b = load_elem(in_type, B, transB ? j * ldb + k : k * ldb + j);
            acc += a * b;
            s += fabs(a) * fabs(b);
        }
        double r = alpha * acc;
        if (beta != 0.0)
            r += beta * load_elem(c_type, C0, i * ldc + j);
        ref[t] = r;
        if (S)
            S[t] = s;
    }
    return ORACLE_OK;
}

/* ---- the definition over a row set x column set ------------------------- */

/* ref / S (each p x q, dense row-major) for rows I[0..p) and columns J[0..q)
 * of C.  I == NULL means rows 0..p-1 (then p must be M); J likewise.  The
 * needed rows of op(A) and columns of op(B) are first decoded into dense
 * double arrays (data staging only); the sum itself is the triple loop,
 * i outermost, k ascending for every (i,j). */
int oracle_gemm_submatrix(int in_type, int c_type, int transA, int transB, int64_t M, int64_t N, int64_t K,
                          double alpha, const void *A, int64_t lda, const void *B, int64_t ldb, double beta,
                          const void *C0, int64_t ldc, int64_t p, const int64_t *I, int64_t q,
                          const int64_t *J, double *ref, double *S)
{
    int rc = check_args(in_type, c_type, transA, transB, M, N, K, lda, ldb, ldc);
    if (rc)
        return rc;
    if (p < 0 || q < 0 || (!I && p != M) || (!J && q != N))
        return ORACLE_BAD_ARG;
    if (p == 0 || q == 0)
        return ORACLE_OK;
    if (!ref || (beta != 0.0 && !C0))
        return ORACLE_BAD_ARG;
    for (int64_t a = 0; I && a < p; ++a)
        if (I[a] < 0 || I[a] >= M)
            return ORACLE_BAD_ARG;
    for (int64_t b = 0; J && b < q; ++b)
        if (J[b] < 0 || J[b] >= N)
            return ORACLE_BAD_ARG;

    size_t ka = (size_t)(K > 0 ? K : 1);
    double *Ad = (double *)malloc(sizeof(double) * (size_t)p * ka); /* p x K */
    double *Bd = (double *)malloc(sizeof(double) * ka * (size_t)q); /* K x q */
    if (!Ad || !Bd) {
        free(Ad);
        free(Bd);
        return ORACLE_NO_MEM;
    }
#pragma omp parallel for schedule(static)
    for (int64_t a = 0; a < p; ++a) {
        int64_t i = I ? I[a] : a;
        for (int64_t k = 0; k < K; ++k)
            Ad[a * K + k] = load_elem(in_type, A, transA ? k * lda + i : i * lda + k);
    }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < K; ++k)
        for (int64_t b = 0; b < q; ++b) {
            int64_t j = J ? J[b] : b;
            Bd[k * q + b] = load_elem(in_type, B, transB ? j * ldb + k : k * ldb + j);
        }

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < p; ++a) {
        double *acc = ref + a * q;
        double *s = S ? S + a * q : NULL;
        for (int64_t b = 0; b < q; ++b)
            acc[b] = 0.0;
        if (s)
            for (int64_t b = 0; b < q; ++b)
                s[b] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double av = Ad[a * K + k];
            const double *brow = Bd + k * q;
            for (int64_t b = 0; b < q; ++b)
                acc[b] += av * brow[b];
            if (s) {
                double aa = fabs(av);
                for (int64_t b = 0; b < q; ++b)
                    s[b] += aa * fabs(brow[b]);
            }
        }
        int64_t i = I ? I[a] : a;
        for (int64_t b = 0; b < q; ++b) {
            int64_t j = J ? J[b] : b;
            double r = alpha * acc[b];
            if (beta != 0.0)
                r += beta * load_elem(c_type, C0, i * ldc + j);
            acc[b] = r;
        }
    }
    free(Ad);
    free(Bd);
    return ORACLE_OK;
}

/* Whole matrix: ref / S are M x N dense row-major. */
int oracle_gemm(int in_type, int c_type, int transA, int transB, int64_t M, int64_t N, int64_t K, double alpha,
                const void *A, int64_t lda, const void *B, int64_t ldb, double beta, const void *C0,
                int64_t ldc, double *ref, double *S)
{
    return oracle_gemm_submatrix(in_type, c_type, transA, transB, M, N, K, alpha, A, lda, B, ldb, beta, C0, ldc,
                                 M, NULL, N, NULL, ref, S);
}

/* ---- fused epilogue tail ---------------------------------------------------- */

/* The library's fused entry point computes act(alpha*op(A)*op(B) + beta*C + bias) with the bias broadcast
 * down the rows; the paper motivates such fusion (sections 1 and 3.2) without defining one.  Here the
 * tail is applied, in fp64, to an already computed `x` (rows x cols, dense): x += bias[col], then
 *   act 0: identity;   act 1: ReLU, max(x, 0);   act 2: GELU, 0.5 x (1 + erf(x / sqrt 2)) = x * Phi(x). */
int oracle_bias_act(double *x, int64_t rows, int64_t cols, const double *bias, int act)
{
    if (rows < 0 || cols < 0 || act < 0 || act > 2 || (rows * cols > 0 && !x))
        return ORACLE_BAD_ARG;
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            double v = x[i * cols + j];
            if (bias)
                v += bias[j];
            if (act == 1)
                v = v > 0.0 ? v : (v == v ? 0.0 : v); /* NaN stays NaN */
            else if (act == 2)
                v = 0.5 * v * (1.0 + erf(v * 0.70710678118654752440));
            x[i * cols + j] = v;
        }
    return ORACLE_OK;
}

/* Residual operand of the fused tail (an addition beyond the paper, like the tail itself): after bias and
 * activation, x(i,j) += R(i,j), with R an M x N row-major matrix of storage type r_type and pitch ldr, decoded
 * exactly; the sum stays in fp64 (the caller rounds once). */
int oracle_residual_add(double *x, int64_t rows, int64_t cols, int r_type, const void *R, int64_t ldr)
{
    if (rows < 0 || cols < 0 || r_type < ORACLE_F16 || r_type > ORACLE_F32 || (rows * cols > 0 && (!x || !R)) || ldr < cols)
        return ORACLE_BAD_ARG;
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            x[i * cols + j] += load_elem(r_type, R, i * ldr + j);
    return ORACLE_OK;
}

size_t oracle_elem_size(int t)
{
    return elem_size(t);
}
