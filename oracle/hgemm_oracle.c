/*
 * hgemm_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, obviously-correct CPU statement of the computation the GPU
 * library performs: half-precision GEMM  C = A * B^T  (paper section 2.1,
 * "HGEMM", with alpha = 1 and beta = 0; the "TN" layout of the paper's
 * Listing 6: A row-major M x K, B stored as N rows of K contiguous halves,
 * C row-major M x N):
 *
 *     C_ref[i][j] = sum_{k=0}^{K-1} f64(A[i][k]) * f64(B[j][k])
 *
 * It plays the part of the CPU reference of the paper's Eq. 1 (section 2.3,
 * "Correctness"), but accumulates in fp64 instead of fp32: every product of two
 * fp16 values is exact in fp64 (22 significand bits), and the fp64 running sum
 * adds at most K * 2^-53 relative error, far below one fp16 ulp.
 *
 * Rules this file keeps:
 *   - a triple loop, k innermost, accumulated left to right; no blocking, no
 *     SIMD intrinsics, no BLAS.  OpenMP splits the rows i across threads, which
 *     does not change any element's summation order.
 *   - its own IEEE binary16 codec written from the format definition
 *     (1 sign, 5 exponent bits with bias 15, 10 fraction bits); no cuda_fp16.h,
 *     no compiler half type, nothing shared with the GPU path.
 *   - fp16 -> fp64 conversion happens inside the loop, through a 65536-entry
 *     table that the codec below fills once.
 *
 * Only tests, the smoke check and the bench's cpu_baseline/reference legs may
 * call into this file.
 *
 * Pins (see tests/test_oracle_*.py): the decoder against all 65536 bit patterns
 * of an independent codec, the encoder on ties / subnormal / overflow
 * boundaries, the loop against exact int64 arithmetic on integer inputs,
 * identity / permutation / rank-1 closed forms, a library fp64 matmul, and
 * exact rational brute force on tiny shapes.
 * Parity unpinned: propagation of Inf/NaN inputs through the loop (unreachable
 * at the library's workloads).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- IEEE 754 binary16 codec ------------------------------------------------ */

/* Value of a binary16 bit pattern: (-1)^s * 2^(e-15) * (1 + f/1024) for
 * 1 <= e <= 30, (-1)^s * 2^-14 * (f/1024) for e == 0, Inf/NaN for e == 31. */
double oracle_f16_bits_to_f64(uint16_t h)
{
    int s = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)f, -24);             /* subnormal or zero: f * 2^-24 */
    } else if (e == 31) {
        v = f ? NAN : INFINITY;
    } else {
        v = ldexp((double)(1024 + f), e - 25); /* (1024+f) * 2^(e-15-10) */
    }
    return s ? -v : v;
}

/* Round a double to the nearest binary16 (ties to even), gradual underflow,
 * overflow to infinity.  Returns the bit pattern. */
uint16_t oracle_f64_to_f16_bits_rne(double x)
{
    uint16_t sign = signbit(x) ? 0x8000u : 0u;
    double a = fabs(x);
    if (isnan(x)) return (uint16_t)(sign | 0x7e00u);
    if (isinf(x)) return (uint16_t)(sign | 0x7c00u);
    if (a == 0.0) return sign;

    int ex;
    (void)frexp(a, &ex);          /* a = m * 2^ex, m in [0.5, 1) => a in [2^(ex-1), 2^ex) */
    int e = ex - 1;               /* floor(log2(a)) */
    if (e < -14) e = -14;         /* subnormal range shares the spacing of 2^-14 */
    /* spacing of binary16 numbers in this binade: 2^(e-10) */
    double q = ldexp(a, 10 - e);  /* a in units of the spacing; exact (power-of-two scaling) */
    double fl = floor(q);
    double r = q - fl;            /* exact: q has at most 53 bits */
    uint64_t n = (uint64_t)fl;
    if (r > 0.5 || (r == 0.5 && (n & 1u))) n += 1;
    /* n is the significand in units of the spacing: < 1024 => subnormal,
     * 1024..2047 => normal with exponent e, 2048 => carries into the next binade */
    if (n == 2048) { n = 1024; e += 1; }
    if (n < 1024) {
        return (uint16_t)(sign | (uint16_t)n);  /* e == -14 here; n may be 0 (underflow to zero) */
    }
    if (e > 15) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | (uint16_t)((e + 15) << 10) | (uint16_t)(n - 1024));
}

void oracle_f64_to_f16_bits_rne_array(int64_t n, const double *x, uint16_t *out)
{
    for (int64_t t = 0; t < n; ++t) out[t] = oracle_f64_to_f16_bits_rne(x[t]);
}

void oracle_f16_bits_to_f64_array(int64_t n, const uint16_t *h, double *out)
{
    for (int64_t t = 0; t < n; ++t) out[t] = oracle_f16_bits_to_f64(h[t]);
}

static double g_decode[65536];
static int g_decode_ready = 0;

static void fill_decode_table(void)
{
    if (g_decode_ready) return;
    for (uint32_t h = 0; h < 65536u; ++h) g_decode[h] = oracle_f16_bits_to_f64((uint16_t)h);
    g_decode_ready = 1;
}

/* ---- the GEMM ------------------------------------------------------------- */

/* Full output.  A: M rows, row stride lda halves; B: N rows, row stride ldb
 * halves; C: M x N doubles, row-major, dense.  Returns the number of threads
 * used. */
int oracle_hgemm_full(int64_t M, int64_t N, int64_t K,
                      const uint16_t *A, int64_t lda,
                      const uint16_t *B, int64_t ldb,
                      double *C)
{
    fill_decode_table();
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#pragma omp parallel for schedule(static)
#endif
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                acc += g_decode[A[i * lda + k]] * g_decode[B[j * ldb + k]];
            }
            C[i * N + j] = acc;
        }
    }
    return threads;
}

/* Sampled output: out[t] = C_ref[ii[t]][jj[t]] for t < n.  ii indexes rows of A,
 * jj rows of B (the caller may pass gathered row subsets and matching indices). */
int oracle_hgemm_sampled(int64_t K,
                         const uint16_t *A, int64_t lda,
                         const uint16_t *B, int64_t ldb,
                         int64_t n, const int64_t *ii, const int64_t *jj,
                         double *out)
{
    fill_decode_table();
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#pragma omp parallel for schedule(static)
#endif
    for (int64_t t = 0; t < n; ++t) {
        const uint16_t *a = A + ii[t] * lda;
        const uint16_t *b = B + jj[t] * ldb;
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            acc += g_decode[a[k]] * g_decode[b[k]];
        }
        out[t] = acc;
    }
    return threads;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
