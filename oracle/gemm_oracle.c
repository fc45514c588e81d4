/*
 * CPU oracle for the dense product C = A * B with 16-bit inputs.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the GPU
 * library is checked against; it shares no code with that library and the
 * library never calls it.
 *
 * What it computes (paper Section 4.1 problem statement, and the "Common"
 * template paragraph around Eq. 2: an M x K matrix times a K x N matrix,
 * products accumulated at higher precision than the inputs and cast once to
 * the 16-bit output type):
 *
 *     C64[i][j] = sum_{k=0}^{K-1} (double)A[i][k] * (double)B[k][j]
 *
 * summed in ascending k in IEEE binary64, and
 *
 *     C16[i][j] = RN-even_16( C64[i][j] )
 *
 * rounded directly from binary64 to binary16 / bfloat16 (no detour through
 * binary32), overflow to +-inf, NaN kept as a quiet NaN.
 *
 * Plain loops, i-k-j order; the only parallelism is OpenMP over output rows.
 * The 16-bit decoders and encoders below are this file's own bit-level code.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F16 0
#define ORACLE_BF16 1
#define ORACLE_ROW_MAJOR 0
#define ORACLE_COL_MAJOR 1

/* ---- 16-bit -> double, exact -------------------------------------------- */

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
double oracle_f16_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)f, -24);              /* zero or subnormal: f * 2^-24 */
    } else if (e == 31) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(f + 1024), e - 25);  /* (1 + f/1024) * 2^(e-15) */
    }
    return sign ? -v : v;
}

/* bfloat16: 1 sign, 8 exponent (bias 127), 7 fraction bits. */
double oracle_bf16_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int f = h & 0x7f;
    double v;
    if (e == 0) {
        v = ldexp((double)f, -133);             /* f * 2^-126 * 2^-7 */
    } else if (e == 255) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(f + 128), e - 134);  /* (1 + f/128) * 2^(e-127) */
    }
    return sign ? -v : v;
}

/* ---- double -> 16-bit, round to nearest even, one rounding ---------------
 * Generic over the format: `fbits` fraction bits, `ebits` exponent bits.
 * Works on the exact binary64 value: scale so that one unit in the last place
 * of the target becomes 1.0, then round the (exactly representable) scaled
 * value to an integer with ties to even.                                     */
static uint16_t encode16(double x, int fbits, int ebits)
{
    int bias = (1 << (ebits - 1)) - 1;
    int emax = bias;                 /* largest normal exponent   */
    int emin = 1 - bias;             /* smallest normal exponent  */
    uint16_t sign = 0;
    uint16_t exp_all = (uint16_t)(((1 << ebits) - 1) << fbits);
    if (isnan(x)) return (uint16_t)(exp_all | (1 << (fbits - 1)));
    if (signbit(x)) { sign = (uint16_t)(1u << (fbits + ebits)); x = -x; }
    if (isinf(x)) return (uint16_t)(sign | exp_all);
    if (x == 0.0) return sign;

    int e;
    (void)frexp(x, &e);              /* x = m * 2^e with m in [0.5, 1) */
    e -= 1;                          /* x = m' * 2^e with m' in [1, 2) */
    if (e < emin) e = emin;          /* subnormal range shares emin's spacing */
    /* one ulp at exponent e is 2^(e - fbits) */
    double scaled = ldexp(x, fbits - e);   /* exact: a power-of-two scaling */
    double fl = floor(scaled);
    double rem = scaled - fl;              /* exact */
    uint64_t q = (uint64_t)fl;
    if (rem > 0.5 || (rem == 0.5 && (q & 1))) q += 1;
    /* q is in [0, 2^(fbits+1)]; q == 2^(fbits+1) means the rounding carried */
    if (q == ((uint64_t)1 << (fbits + 1))) { q >>= 1; e += 1; }
    if (q < ((uint64_t)1 << fbits)) {
        /* subnormal (or zero after rounding): biased exponent field 0 */
        return (uint16_t)(sign | (uint16_t)q);
    }
    if (e > emax) return (uint16_t)(sign | exp_all);   /* overflow -> inf */
    return (uint16_t)(sign | (uint16_t)((e + bias) << fbits) |
                      (uint16_t)(q - ((uint64_t)1 << fbits)));
}

uint16_t oracle_f64_to_f16(double x)  { return encode16(x, 10, 5); }
uint16_t oracle_f64_to_bf16(double x) { return encode16(x, 7, 8); }

double oracle_decode16(uint16_t h, int dtype)
{
    return dtype == ORACLE_BF16 ? oracle_bf16_to_f64(h) : oracle_f16_to_f64(h);
}
uint16_t oracle_encode16(double x, int dtype)
{
    return dtype == ORACLE_BF16 ? oracle_f64_to_bf16(x) : oracle_f64_to_f16(x);
}

void oracle_decode16_array(const uint16_t* in, double* out, size_t n, int dtype)
{
    for (size_t i = 0; i < n; ++i) out[i] = oracle_decode16(in[i], dtype);
}
void oracle_encode16_array(const double* in, uint16_t* out, size_t n, int dtype)
{
    for (size_t i = 0; i < n; ++i) out[i] = oracle_encode16(in[i], dtype);
}

/* ---- the product --------------------------------------------------------- */

/* Element (i,k) of A (M x K) and (k,j) of B (K x N), dense storage:
 * row-major A has leading dimension K, column-major A has leading dimension M;
 * row-major B has leading dimension N, column-major B has leading dimension K. */
static inline size_t idxA(int64_t i, int64_t k, int64_t M, int64_t K, int layoutA)
{
    return layoutA == ORACLE_ROW_MAJOR ? (size_t)i * (size_t)K + (size_t)k
                                       : (size_t)k * (size_t)M + (size_t)i;
}
static inline size_t idxB(int64_t k, int64_t j, int64_t K, int64_t N, int layoutB)
{
    return layoutB == ORACLE_ROW_MAJOR ? (size_t)k * (size_t)N + (size_t)j
                                       : (size_t)j * (size_t)K + (size_t)k;
}

/*
 * Rows rows[0..nrows) of the product.  C64 (nrows x N, row-major, may be NULL)
 * receives the binary64 sums, C16 (nrows x N, may be NULL) their single
 * rounding to the 16-bit type.  rows == NULL means rows 0..nrows-1.
 * Returns 0, or -1 on a bad argument.
 *
 * The decode of a 16-bit word goes through a 65,536-entry table filled by the
 * decoders above, so the inner loop is one table read, one multiply, one add.
 */
int oracle_gemm_rows(int64_t M, int64_t N, int64_t K, int dtype, int layoutA, int layoutB,
                     const uint16_t* A, const uint16_t* B,
                     const int64_t* rows, int64_t nrows,
                     double* C64, uint16_t* C16, int nthreads)
{
    if (M < 0 || N < 0 || K < 0 || nrows < 0) return -1;
    if (dtype != ORACLE_F16 && dtype != ORACLE_BF16) return -1;
    if (nrows == 0 || N == 0) return 0;

    static double lut[2][65536];
    static int lut_ready[2] = {0, 0};
#ifdef _OPENMP
#pragma omp critical(oracle_lut)
#endif
    {
        if (!lut_ready[dtype]) {
            for (uint32_t h = 0; h < 65536; ++h) lut[dtype][h] = oracle_decode16((uint16_t)h, dtype);
            lut_ready[dtype] = 1;
        }
    }
    const double* T = lut[dtype];
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t i = rows ? rows[r] : r;
        if (i < 0 || i >= M) return -1;
    }

#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1) num_threads(nthreads)
#endif
    for (int64_t r = 0; r < nrows; ++r) {
        int64_t i = rows ? rows[r] : r;
        /* accumulate row i in a private binary64 buffer */
        double* c = C64 ? C64 + (size_t)r * (size_t)N : NULL;
        double* tmp = NULL;
        if (!c) {
            tmp = (double*)__builtin_malloc((size_t)N * sizeof(double));
            c = tmp;
        }
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double a = T[A[idxA(i, k, M, K, layoutA)]];
            if (layoutB == ORACLE_ROW_MAJOR) {
                const uint16_t* brow = B + (size_t)k * (size_t)N;
                for (int64_t j = 0; j < N; ++j) c[j] += a * T[brow[j]];
            } else {
                for (int64_t j = 0; j < N; ++j) c[j] += a * T[B[idxB(k, j, K, N, layoutB)]];
            }
        }
        if (C16) {
            uint16_t* o = C16 + (size_t)r * (size_t)N;
            for (int64_t j = 0; j < N; ++j) o[j] = oracle_encode16(c[j], dtype);
        }
        if (tmp) __builtin_free(tmp);
    }
    return 0;
}

/* Whole product: every row. */
int oracle_gemm(int64_t M, int64_t N, int64_t K, int dtype, int layoutA, int layoutB,
                const uint16_t* A, const uint16_t* B, double* C64, uint16_t* C16, int nthreads)
{
    return oracle_gemm_rows(M, N, K, dtype, layoutA, layoutB, A, B, NULL, M, C64, C16, nthreads);
}

/*
 * Normwise comparison used by the acceptance bar: accumulates
 *   num += (decode(Cgot[i]) - Cref[i])^2 ,  den += Cref[i]^2
 * in binary64 over n elements.  Non-finite differences are counted in *nonfinite.
 */
void oracle_fro_accumulate(const uint16_t* Cgot, const double* Cref, size_t n, int dtype,
                           double* num, double* den, int64_t* nonfinite)
{
    double s = 0.0, t = 0.0;
    int64_t bad = 0;
    for (size_t i = 0; i < n; ++i) {
        double g = oracle_decode16(Cgot[i], dtype);
        double d = g - Cref[i];
        if (!isfinite(d)) { ++bad; continue; }
        s += d * d;
        t += Cref[i] * Cref[i];
    }
    *num += s; *den += t; *nonfinite += bad;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- the fused-add operator (an extension; the functions above are untouched) ----------- */

/*
 * Rows rows[0..nrows) of   Out = alpha * (A * B) + beta * D,
 * the AddMM operator the paper lists beside MatMul among the operators it replaces
 * (Section 6.5).  The product is the binary64 sum of oracle_gemm_rows (ascending k); alpha and
 * beta are binary64 (the caller passes the exact values of the binary32 scalars the library
 * takes); D holds 16-bit words of the same type as A and B and is either a full M x N row-major
 * matrix (d_is_vector == 0) or one row of N values added to every output row (d_is_vector != 0,
 * a bias).  One multiplication and one addition per term, in binary64, then ONE rounding to the
 * 16-bit type: out64 = alpha * sum + beta * d.  O64 / O16 as in oracle_gemm_rows.
 */
int oracle_addmm_rows(int64_t M, int64_t N, int64_t K, int dtype, int layoutA, int layoutB,
                      const uint16_t* A, const uint16_t* B, const uint16_t* D, int d_is_vector,
                      double alpha, double beta,
                      const int64_t* rows, int64_t nrows,
                      double* O64, uint16_t* O16, int nthreads)
{
    if (nrows < 0 || N < 0 || !D) return -1;
    if (nrows == 0 || N == 0) return 0;
    double* sum = (double*)__builtin_malloc((size_t)nrows * (size_t)N * sizeof(double));
    if (!sum) return -1;
    int rc = oracle_gemm_rows(M, N, K, dtype, layoutA, layoutB, A, B, rows, nrows, sum, NULL, nthreads);
    if (rc == 0) {
        for (int64_t r = 0; r < nrows; ++r) {
            int64_t i = rows ? rows[r] : r;
            for (int64_t j = 0; j < N; ++j) {
                double d = oracle_decode16(d_is_vector ? D[j] : D[(size_t)i * (size_t)N + (size_t)j], dtype);
                double v = alpha * sum[(size_t)r * (size_t)N + (size_t)j] + beta * d;
                if (O64) O64[(size_t)r * (size_t)N + (size_t)j] = v;
                if (O16) O16[(size_t)r * (size_t)N + (size_t)j] = oracle_encode16(v, dtype);
            }
        }
    }
    __builtin_free(sum);
    return rc;
}
