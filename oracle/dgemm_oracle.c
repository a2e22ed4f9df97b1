/*
 * dgemm_oracle.c -- CPU oracle for C += A*B in IEEE binary64 (TEST INFRASTRUCTURE ONLY).
 *
 * See dgemm_oracle.h for the semantics and the list of pins. Build with
 *   gcc -O2 -fno-fast-math -ffp-contract=off -fopenmp -shared -fPIC
 * so that the compiler neither reassociates sums nor contracts a*b+c into an fma: every
 * output element is the running sum c = c + a*b over ascending k, started from the incoming
 * C value, with the product and the sum each rounded once (the operation C += A*B of the
 * paper's Section 2.1).
 *
 * Nothing here is blocked, packed, unrolled or otherwise tuned, on purpose.
 */
#include "dgemm_oracle.h"

#include <math.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/*
 * The definition. Each entry is one inner product added to what C already holds: a scalar
 * starts at C[i][j], takes the K products in ascending k, and is written back once. Nothing
 * else touches C[i][j] meanwhile, so keeping the sum in a scalar rounds exactly as updating
 * C in memory after every k would.
 */
void dgemm_oracle_ijk(int64_t M, int64_t N, int64_t K,
                      const double *A, int64_t lda,
                      const double *B, int64_t ldb,
                      double *C, int64_t ldc)
{
    for (int64_t i = 0; i < M; ++i) {
        const double *arow = A + i * lda;
        for (int64_t j = 0; j < N; ++j) {
            double acc = C[i * ldc + j];
            for (int64_t k = 0; k < K; ++k) {
                acc = acc + arow[k] * B[k * ldb + j]; /* -ffp-contract=off: two roundings */
            }
            C[i * ldc + j] = acc;
        }
    }
}

/*
 * Interchanged order i, k, j. For a fixed (i,j) the updates still happen for k = 0, 1, ...,
 * K-1 in that order and each one is c = c + a*b with two roundings, so every element sees
 * the operation sequence of the definition. Rows are independent: one row per OpenMP task.
 */
void dgemm_oracle_ikj(int64_t M, int64_t N, int64_t K,
                      const double *A, int64_t lda,
                      const double *B, int64_t ldb,
                      double *C, int64_t ldc, int threads)
{
#ifdef _OPENMP
    int nt = threads > 0 ? threads : omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nt)
#else
    (void)threads;
#endif
    for (int64_t i = 0; i < M; ++i) {
        double *c = C + i * ldc;
        for (int64_t k = 0; k < K; ++k) {
            const double a = A[i * lda + k];
            const double *b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) {
                c[j] = c[j] + a * b[j]; /* -ffp-contract=off: multiply, then add */
            }
        }
    }
}

void dgemm_oracle_entries(int64_t K,
                          const double *A, int64_t lda,
                          const double *B, int64_t ldb,
                          const double *Cin, int64_t ldc,
                          int64_t nsamples, const int64_t *ii, const int64_t *jj,
                          int absolute, double *out, int threads)
{
#ifdef _OPENMP
    int nt = threads > 0 ? threads : omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nt)
#else
    (void)threads;
#endif
    for (int64_t s = 0; s < nsamples; ++s) {
        const int64_t i = ii[s], j = jj[s];
        double c = Cin ? Cin[i * ldc + j] : 0.0;
        if (absolute) c = fabs(c);
        for (int64_t k = 0; k < K; ++k) {
            double a = A[i * lda + k];
            double b = B[k * ldb + j];
            if (absolute) { a = fabs(a); b = fabs(b); }
            c = c + a * b; /* two roundings, as above */
        }
        out[s] = c;
    }
}

void dgemm_oracle_general(int transa, int transb, int64_t M, int64_t N, int64_t K,
                          double alpha, const double *A, int64_t lda,
                          const double *B, int64_t ldb,
                          double beta, double *C, int64_t ldc, int threads)
{
    const int product = (alpha != 0.0) && K > 0;
#ifdef _OPENMP
    int nt = threads > 0 ? threads : omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nt)
#else
    (void)threads;
#endif
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            if (product) {
                for (int64_t k = 0; k < K; ++k) {
                    const double a = transa ? A[k * lda + i] : A[i * lda + k];
                    const double b = transb ? B[j * ldb + k] : B[k * ldb + j];
                    s = s + a * b; /* multiply, then add (no contraction) */
                }
            }
            const double as = product ? alpha * s : 0.0;
            if (beta == 0.0) {
                C[i * ldc + j] = as;
            } else {
                const double bc = beta * C[i * ldc + j];
                C[i * ldc + j] = as + bc;
            }
        }
    }
}

void sgemm_oracle_ijk(int64_t M, int64_t N, int64_t K,
                      const float *A, int64_t lda,
                      const float *B, int64_t ldb,
                      float *C, int64_t ldc)
{
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            float c = C[i * ldc + j];
            for (int64_t k = 0; k < K; ++k) {
                const float prod = A[i * lda + k] * B[k * ldb + j]; /* rounded to binary32 */
                c = c + prod;                                       /* rounded to binary32 */
            }
            C[i * ldc + j] = c;
        }
    }
}

void sgemm_oracle_ikj(int64_t M, int64_t N, int64_t K,
                      const float *A, int64_t lda,
                      const float *B, int64_t ldb,
                      float *C, int64_t ldc, int threads)
{
#ifdef _OPENMP
    int nt = threads > 0 ? threads : omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nt)
#else
    (void)threads;
#endif
    for (int64_t i = 0; i < M; ++i) {
        float *c = C + i * ldc;
        for (int64_t k = 0; k < K; ++k) {
            const float a = A[i * lda + k];
            const float *b = B + k * ldb;
            for (int64_t j = 0; j < N; ++j) {
                const float prod = a * b[j];
                c[j] = c[j] + prod;
            }
        }
    }
}

void sgemm_oracle_entries(int64_t K,
                          const float *A, int64_t lda,
                          const float *B, int64_t ldb,
                          const float *Cin, int64_t ldc,
                          int64_t nsamples, const int64_t *ii, const int64_t *jj,
                          float *out, int threads)
{
#ifdef _OPENMP
    int nt = threads > 0 ? threads : omp_get_max_threads();
#pragma omp parallel for schedule(static) num_threads(nt)
#else
    (void)threads;
#endif
    for (int64_t s = 0; s < nsamples; ++s) {
        const int64_t i = ii[s], j = jj[s];
        float c = Cin ? Cin[i * ldc + j] : 0.0f;
        for (int64_t k = 0; k < K; ++k) {
            const float prod = A[i * lda + k] * B[k * ldb + j];
            c = c + prod;
        }
        out[s] = c;
    }
}

int dgemm_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
