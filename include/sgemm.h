/*
 * sgemm.h -- C ABI of the single-precision entry point of libdgemm (NVIDIA B200, sm_100a).
 *
 * The paper's second workload (Section 2.13 "SGEMM performance"): the same operation with every
 * f64 replaced by f32, C += A*B on row-major binary32 matrices, alpha = beta = 1. The library
 * computes it in exact binary32 arithmetic (fused multiply-adds on the FP32 pipe); the reduced-
 * precision tensor-core formats (TF32 and narrower) change the result and are not used.
 *
 * Plain C types only; status codes are those of dgemm.h.
 */
#ifndef SGEMM_H
#define SGEMM_H

#include <stdint.h>

#include "dgemm.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * C[i][j] += sum_k A[i][k] * B[k][j] for 0 <= i < M, 0 <= j < N, in binary32.
 *
 *   A  device pointer, M x K floats, row-major, leading dimension lda >= max(1,K); read only
 *   B  device pointer, K x N floats, row-major, leading dimension ldb >= max(1,N); read only
 *   C  device pointer, M x N floats, row-major, leading dimension ldc >= max(1,N); read and written
 *   stream  a cudaStream_t passed as void*; NULL is the legacy default stream
 *
 * Buffers live on the current CUDA device and stay owned by the caller. Asynchronous: work is
 * enqueued on `stream`. Each entry's sum is accumulated from +0 in ascending k with fused
 * multiply-adds, the incoming C value is added last; the result equals the definition's within
 * 2*K*2^-24*(|C| + |A||B|)_ij and exactly when every partial sum is representable (small-integer
 * data). Only the logical M x K, K x N and M x N parts are read, only C[i<M][j<N] is written.
 *
 * M == 0 or N == 0: DGEMM_OK without inspecting pointers. K == 0: DGEMM_OK, C untouched.
 * Pointers must be 4-byte aligned (DGEMM_ERR_ALIGN); C must not overlap A or B (DGEMM_ERR_ALIAS).
 * Operands that the tensor-copy engine cannot address (A or B not 16-byte aligned, or a leading
 * dimension that is not a multiple of 4) are first copied into library-owned scratch memory (grown
 * on demand with a synchronising cudaMalloc). That buffer and the workspace of the partial tiles
 * are leased per call exactly as for dgemm_f64, so calls may be in flight on several streams at
 * once. Other error codes as for dgemm_f64.
 */
DGEMM_API int sgemm_f32(int64_t M, int64_t N, int64_t K,
                        const float *A, int64_t lda,
                        const float *B, int64_t ldb,
                        float *C, int64_t ldc,
                        void *stream);

/* Synchronises `stream`, then reads and clears the device status word of the sgemm kernels
 * (DGEMM_OK, DGEMM_ERR_TIMEOUT if a bounded wait inside a kernel gave up, DGEMM_ERR_CUDA). */
DGEMM_API int sgemm_last_device_status(void *stream);

#ifdef __cplusplus
}
#endif
#endif
