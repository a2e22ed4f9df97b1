/*
 * dgemm_oracle.h -- CPU oracle for C += A*B in IEEE binary64 (TEST INFRASTRUCTURE ONLY).
 *
 * This is the slow, obviously-correct definition that the GPU library is checked against.
 * It is used only by the test-suite, by the smoke check and by the benchmark's CPU-baseline
 * leg. It shares no source, header, table or helper with the CUDA path and is never on the
 * product path.
 *
 * Semantics follow the paper's problem statement (Section 2.1 "Affine Ops", the naive
 * three-deep nest, and Section 2.2 "MemRefs", identity layout map): three distinct row-major
 * buffers, element (i,j) of a matrix with leading dimension ld lives at base[i*ld + j], and
 *
 *     C[i][j] <- C[i][j] + sum_{k=0..K-1} A[i][k] * B[k][j]        (alpha = beta = 1)
 *
 * evaluated for each (i,j) as c = c + a*b with k ascending, the product and the sum each
 * rounded once (no fused multiply-add), round to nearest even. Columns j >= N of C (row padding) are never written; columns k >= K of A and j >= N
 * of B are never read.
 *
 * Parity pins (tests/test_oracle_pins.py): the all-ones driver input of the paper
 * (every entry becomes 1 + K), identity and permutation operands, rank-1 products, int64
 * brute force on tiny shapes, exact rational recomputation within the textbook error bound,
 * loop-order identity, K-split invariance, transpose symmetry, linearity, padding canaries and
 * a BLAS cross-check. No function here is "parity unpinned".
 */
#ifndef DGEMM_ORACLE_H
#define DGEMM_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* The definition itself: loops i, j, k, one running sum per entry. Single-threaded. Host pointers. */
void dgemm_oracle_ijk(int64_t M, int64_t N, int64_t K,
                      const double *A, int64_t lda,
                      const double *B, int64_t ldb,
                      double *C, int64_t ldc);

/*
 * Loop interchange i, k, j (the textbook interchange the paper mentions when discussing what
 * compilers do to the naive nest, Section 1.3.1). For every (i,j) the same operations are
 * applied in the same k order, so the result is bit-identical to dgemm_oracle_ijk. Rows of C
 * are independent and are distributed over `threads` OpenMP threads (<= 0: library default).
 */
void dgemm_oracle_ikj(int64_t M, int64_t N, int64_t K,
                      const double *A, int64_t lda,
                      const double *B, int64_t ldb,
                      double *C, int64_t ldc, int threads);

/*
 * Sampled entries by the definition: out[s] = Cin[ii[s]][jj[s]] + sum_k A[ii[s]][k]*B[k][jj[s]],
 * k ascending, unfused. Cin may be NULL (treated as +0). If `absolute` is non-zero the
 * magnitudes |Cin|, |A|, |B| are used instead (this yields the (|C|+|A||B|)_ij error-bound
 * scale). Entries are independent and distributed over OpenMP threads.
 */
void dgemm_oracle_entries(int64_t K,
                          const double *A, int64_t lda,
                          const double *B, int64_t ldb,
                          const double *Cin, int64_t ldc,
                          int64_t nsamples, const int64_t *ii, const int64_t *jj,
                          int absolute, double *out, int threads);

/*
 * General form (Section 2.15, "Other questions": the scalars and the transposed layouts that the
 * paper names but sets to alpha = beta = 1, no transposition):
 *
 *     C[i][j] <- alpha * s_ij + beta * C[i][j],   s_ij = sum_{k} opA(i,k) * opB(k,j)
 *
 * opA(i,k) = A[i*lda + k] (transa == 0) or A[k*lda + i] (transa != 0, A stored K x M);
 * opB(k,j) = B[k*ldb + j] (transb == 0) or B[j*ldb + k] (transb != 0, B stored N x K).
 * s_ij starts from +0 and takes k ascending with a rounded multiply and a rounded add; then one
 * multiply by alpha, one by beta, one add. beta == 0: the old C is not read and the result is
 * alpha * s_ij (a NaN in C does not survive). alpha == 0 or K == 0: A and B are not read.
 * Loops i, j, k; rows over OpenMP threads. Pinned by tests/test_oracle_pins.py (integer brute
 * force with transposes, exact rationals, NaN rules, reduction to the plain definition).
 */
void dgemm_oracle_general(int transa, int transb, int64_t M, int64_t N, int64_t K,
                          double alpha, const double *A, int64_t lda,
                          const double *B, int64_t ldb,
                          double beta, double *C, int64_t ldc, int threads);

/*
 * Single precision (Section 2.13 "SGEMM performance": the same nest with f64 replaced by f32).
 * C[i][j] <- C[i][j] + sum_k A[i][k]*B[k][j] evaluated in IEEE binary32: for each (i,j), k
 * ascending, c = c + a*b with a rounded binary32 multiply followed by a rounded binary32 add (no
 * contraction, no wider intermediate). sgemm_oracle_ijk is the definition (loops i, j, k, single
 * thread); sgemm_oracle_ikj is the interchange over OpenMP rows, bit-identical to it.
 * sgemm_oracle_entries recomputes sampled entries the same way (Cin may be NULL = +0).
 * Pinned by tests/test_oracle_pins.py: all-ones input (1 + K), int brute force, exact rationals
 * within the binary32 bound, a case where binary64 accumulation would give another answer,
 * loop-order identity, padding canaries.
 */
void sgemm_oracle_ijk(int64_t M, int64_t N, int64_t K,
                      const float *A, int64_t lda,
                      const float *B, int64_t ldb,
                      float *C, int64_t ldc);
void sgemm_oracle_ikj(int64_t M, int64_t N, int64_t K,
                      const float *A, int64_t lda,
                      const float *B, int64_t ldb,
                      float *C, int64_t ldc, int threads);
void sgemm_oracle_entries(int64_t K,
                          const float *A, int64_t lda,
                          const float *B, int64_t ldb,
                          const float *Cin, int64_t ldc,
                          int64_t nsamples, const int64_t *ii, const int64_t *jj,
                          float *out, int threads);

/* Number of OpenMP threads a call with threads <= 0 would use. */
int dgemm_oracle_max_threads(void);

#ifdef __cplusplus
}
#endif
#endif
