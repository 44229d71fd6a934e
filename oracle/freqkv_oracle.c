/*
 * FreqKV compression oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what one compression of a KV-cache
 * matrix computes, written from the paper's definitions:
 *
 *   step 1  orthonormal DCT-II along the token axis        (Appendix A, first equation)
 *   step 2  keep the L lowest-frequency components         (Section 3.3, "retaining ratio")
 *   step 3  L-point inverse DCT of the kept components     (Appendix A, second equation,
 *                                                           with N := L, Appendix F.5)
 *   step 4  rescale by sqrt(L/N)                           (Section 3.3, Eq. 3)
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call
 * this file.  It shares no code, tables or headers with the CUDA path.
 *
 * Every routine works on one matrix stored token-major: x[n*d + c] is token n,
 * channel c.  All sums are the defining cosine sums, accumulated in fp64, with
 * no blocking, recursion or fast transform.  The cosine argument
 * pi*t*(2n+1)/(2N) is reduced exactly in integers, k = t*(2n+1) mod 4N, so the
 * value comes from a 4N-entry table of cos(pi*k/(2N)) and the oracle's own
 * error stays at the level of fp64 rounding.
 *
 * Parity pins (tests/test_oracle_pins.py): library DCT cross-check, identity at
 * L = N, constant sequence, Parseval, single-cosine resampling, brute-force
 * matrices on tiny lengths, linearity.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef M_PI
#define M_PI 3.14159265358979323846
#endif

/* cos(pi*k/(2N)) for k = 0 .. 4N-1 (one full period of the DCT-II phase). */
static double *cosine_table(int64_t N)
{
    double *tab = (double *)malloc((size_t)(4 * N) * sizeof(double));
    if (!tab) return NULL;
    for (int64_t k = 0; k < 4 * N; ++k) tab[k] = cos(M_PI * (double)k / (2.0 * (double)N));
    return tab;
}

/* alpha_t of Appendix A: sqrt(1/N) for t = 0, sqrt(2/N) otherwise. */
static double alpha(int64_t t, int64_t N)
{
    return t == 0 ? sqrt(1.0 / (double)N) : sqrt(2.0 / (double)N);
}

/*
 * Appendix A, DCT-II:  z_t = alpha_t * sum_{n<N} x_n cos[pi t (2n+1) / (2N)],
 * for t = 0 .. n_out-1 (n_out <= N; n_out < N is the truncation of Section 3.3).
 * x: N x d, z: n_out x d.  Returns 0, or -1 on allocation failure / bad sizes.
 */
int freqkv_oracle_dct2(const double *x, int64_t N, int64_t d, int64_t n_out, double *z)
{
    if (N <= 0 || d <= 0 || n_out < 0 || n_out > N) return -1;
    double *tab = cosine_table(N);
    if (!tab) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n_out; ++t) {
        double *zt = z + t * d;
        for (int64_t c = 0; c < d; ++c) zt[c] = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            const double w = tab[(t * (2 * n + 1)) % (4 * N)];
            const double *xn = x + n * d;
            for (int64_t c = 0; c < d; ++c) zt[c] += w * xn[c];
        }
        const double a = alpha(t, N);
        for (int64_t c = 0; c < d; ++c) zt[c] *= a;
    }
    free(tab);
    return 0;
}

/*
 * Appendix A, inverse DCT of length L:
 *   y_m = sum_{t<L} alpha_t z_t cos[pi t (2m+1) / (2L)],  m = 0 .. L-1,
 * alpha_t built from L (the kept components are normalised by sqrt(L)).
 * z: L x d, y: L x d.
 */
int freqkv_oracle_idct(const double *z, int64_t L, int64_t d, double *y)
{
    if (L <= 0 || d <= 0) return -1;
    double *tab = cosine_table(L);
    if (!tab) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < L; ++m) {
        double *ym = y + m * d;
        for (int64_t c = 0; c < d; ++c) ym[c] = 0.0;
        for (int64_t t = 0; t < L; ++t) {
            const double w = alpha(t, L) * tab[(t * (2 * m + 1)) % (4 * L)];
            const double *zt = z + t * d;
            for (int64_t c = 0; c < d; ++c) ym[c] += w * zt[c];
        }
    }
    free(tab);
    return 0;
}

/*
 * One compression of one matrix (Section 3.3, Eq. 2-3):
 *   y = sqrt(L/N) * IDCT_L( DCT_N(x)[0:L] ).
 * x: N x d (the non-sink rows of the cache), y: L x d.  L = 0 writes nothing.
 */
int freqkv_oracle_compress(const double *x, int64_t N, int64_t L, int64_t d, double *y)
{
    if (N <= 0 || d <= 0 || L < 0 || L > N) return -1;
    if (L == 0) return 0;
    double *z = (double *)malloc((size_t)(L * d) * sizeof(double));
    if (!z) return -1;
    int rc = freqkv_oracle_dct2(x, N, d, L, z);   /* steps 1-2 */
    if (rc == 0) rc = freqkv_oracle_idct(z, L, d, y); /* step 3 */
    if (rc == 0) {
        const double s = sqrt((double)L / (double)N); /* step 4 */
        for (int64_t i = 0; i < L * d; ++i) y[i] *= s;
    }
    free(z);
    return rc;
}

/* Threads the parallel loops above will use (1 when built without OpenMP). */
int freqkv_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
