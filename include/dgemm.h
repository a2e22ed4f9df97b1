/*
 * dgemm.h -- C ABI of libdgemm: double-precision C += A*B for NVIDIA B200 (sm_100a).
 *
 * The operation is the one the paper studies throughout (Section 2.1 "Affine Ops": the
 * comment and body of the naive nest, "C += A * B" on f64 operands; Section 2.15, question 4:
 * alpha = beta = 1 is assumed). Matrices are row-major with the identity layout map of
 * Section 2.2 "MemRefs": element (i,j) of a matrix with leading dimension ld lives at
 * base[i*ld + j]; a leading dimension larger than the row length expresses the padded layout
 * (d0,d1) -> (d0*ld + d1) of Section 2.11, whose padding can never be accessed.
 *
 * Plain C types only. All functions return a dgemm_status (0 = success, negative = error)
 * unless stated otherwise. Error returns never launch work.
 */
#ifndef DGEMM_H
#define DGEMM_H

#include <stdint.h>

#if defined(__GNUC__)
#define DGEMM_API __attribute__((visibility("default")))
#else
#define DGEMM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DGEMM_OK = 0,
  DGEMM_ERR_BAD_DIM = -1, /* M, N or K < 0, or a dimension beyond 2^31-1 rows/cols            */
  DGEMM_ERR_BAD_LD = -2,  /* lda < max(1,K), ldb < max(1,N) or ldc < max(1,N)                  */
  DGEMM_ERR_NULL = -3,    /* a needed pointer is NULL                                          */
  DGEMM_ERR_ALIGN = -4,   /* a pointer is not 8-byte aligned                                   */
  DGEMM_ERR_ALIAS = -5,   /* the byte range of C overlaps that of A or B                       */
  DGEMM_ERR_DEVICE = -6,  /* no CUDA device, or the current device is not compute capability 10 */
  DGEMM_ERR_CUDA = -7,    /* a CUDA runtime/driver call failed (launch, copy, allocation)      */
  DGEMM_ERR_TIMEOUT = -8, /* a bounded device-side wait gave up (device status word)           */
  DGEMM_ERR_VARIANT = -9, /* unknown variant, or the forced variant cannot run these operands  */
  DGEMM_ERR_SIZE = -10    /* a fixed-capacity entry point was given a problem beyond its limit */
} dgemm_status;

/* Kernel variants (dgemm_set_variant). The ladder mirrors the paper's step-by-step journey
 * (Sections 2.3-2.9): a naive nest first, then tiling + staging ("packing") + register tiling. */
enum {
  DGEMM_VARIANT_AUTO = -1,   /* choose by operand alignment and problem shape (default)         */
  DGEMM_VARIANT_NAIVE = 0,   /* one thread per C element, k sequential (the naive nest on a GPU) */
  DGEMM_VARIANT_TMA = 1,     /* DMMA pipeline, operand tiles staged by TMA; needs 16-byte aligned
                                A and B base pointers and even lda, ldb                          */
  DGEMM_VARIANT_GENERIC = 2, /* same pipeline, tiles staged by 8-byte asynchronous copies; any
                                8-byte aligned operands and any leading dimensions               */
  DGEMM_VARIANT_TMA_WS = 3,     /* as TMA, with a separate producer warpgroup (warp-specialised) and a
                                   software-pipelined consumer loop                              */
  DGEMM_VARIANT_GENERIC_WS = 4, /* as GENERIC, with a separate producer warpgroup                 */
  DGEMM_VARIANT_TMA_CLUSTER = 5, /* as TMA on 64 x 128 tiles, K cut over the 1, 2, 4 or 8 CTAs of a
                                    thread-block cluster, partial tiles added through distributed shared
                                    memory: one launch, no workspace; what AUTO uses below one wave of tiles */
  DGEMM_VARIANT_GENERIC_CLUSTER = 6, /* as TMA_CLUSTER with the GENERIC staging: any alignment          */
  DGEMM_VARIANT_SMEM = 7,        /* ladder rung: tiles of A and B in shared memory, one C element per thread,
                                    no register tile (tiling + packing before unroll-and-jam, Sections 2.4-2.6) */
  DGEMM_VARIANT_TMA_DFMA = 8,    /* micro-kernel swap (Section 2.12): the TMA variant's staging, pipeline, raster
                                    and epilogue on 64 x 128 tiles, with plain FP64 fused multiply-adds on an
                                    8 x 8 register tile per thread in place of the tensor-core MMAs */
  DGEMM_VARIANT_GENERIC_DFMA = 9, /* the same inner kernel under the GENERIC staging: any alignment          */
  DGEMM_VARIANT_TMA_WS_BULK = 10, /* as TMA_WS on 128 x 128 tiles with five stages and the epilogue done by the
                                    copy engine: the accumulators go to a tile buffer in shared memory and
                                    leave row by row as bulk reduces (add) into C, or bulk stores when beta == 0;
                                    C is never loaded into the SM. Needs, besides the TMA conditions, a
                                    16-byte aligned C with even ldc and beta == 0 or 1. What AUTO uses for
                                    large problems with a short K (rank-k updates)                        */
  DGEMM_VARIANT_COUNT = 11
};

/*
 * C[i][j] += sum_k A[i][k] * B[k][j] for 0 <= i < M, 0 <= j < N (Section 2.1, naive nest;
 * alpha = beta = 1, Section 2.15).
 *
 *   A  device pointer, M x K, row-major, leading dimension lda >= max(1,K); read only
 *   B  device pointer, K x N, row-major, leading dimension ldb >= max(1,N); read only
 *   C  device pointer, M x N, row-major, leading dimension ldc >= max(1,N); read and written
 *   stream  a cudaStream_t passed as void*; NULL is the legacy default stream
 *
 * All three buffers live on the current CUDA device and stay owned by the caller; the library
 * neither retains nor frees them. The call is asynchronous: work is enqueued on `stream` and
 * the function returns without synchronising. Arithmetic is IEEE binary64 with fused
 * multiply-adds, round to nearest even; each entry's sum is accumulated from +0 in ascending
 * k (inside one k-split) and the incoming C value is added last, so the result equals the
 * definition's within 2*K*2^-53*(|A||B|)_ij and exactly when every partial sum is exactly
 * representable (e.g. small-integer data).
 *
 * Only A[i][k<K], B[k][j<N] and C[i][j<N] are ever read and only C[i<M][j<N] is written:
 * padding beyond the logical row is neither read into the result nor modified.
 * M == 0 or N == 0: returns DGEMM_OK without inspecting pointers. K == 0: returns DGEMM_OK and
 * leaves C untouched. A and B may alias each other; C must not overlap A or B (checked on byte
 * ranges, DGEMM_ERR_ALIAS). Pointers must be 8-byte aligned; a faster path is taken when A and
 * B are 16-byte aligned with even lda and ldb.
 *
 * Operands that the tensor-copy engine cannot address (A or B not 16-byte aligned, or an odd
 * leading dimension) are, when the problem is large enough for the copy to be cheap next to the
 * arithmetic, first packed into library-owned scratch memory (grown on demand, at most 2 GiB
 * per problem); smaller ones are staged directly with 8-byte copies. Problems with few output
 * tiles split K over several thread blocks; their partial sums go through a library-owned
 * workspace of 80 MiB.
 *
 * Concurrency: calls may be made from several host threads and may be in flight on several
 * streams at once. The scratch memory above is leased per call: a call on a stream never shares
 * its lease with a call still in flight on another stream (calls on one stream run in stream
 * order and reuse one lease). A device holds at most four leases; with more streams than that
 * in flight, a call first makes its stream wait for the least recently used lease's last user.
 * Leases are allocated on first need with a synchronising cudaMalloc: make the first call on a
 * stream outside stream capture. As long as all calls on a device come from one stream nothing
 * else synchronises; the first call on a second stream synchronises the device once. Calls
 * recorded into a CUDA graph use the lease their stream had at capture time; replays of the graph
 * are not covered by the guarantee above and must not overlap other calls that use scratch.
 *
 * The kernels are launched with programmatic stream serialization: their thread blocks may be
 * scheduled while the previous kernel in `stream` is finishing, but they wait for its completion
 * (and the visibility of its writes) before they touch global memory, so stream order holds.
 */
DGEMM_API int dgemm_f64(int64_t M, int64_t N, int64_t K,
              const double *A, int64_t lda,
              const double *B, int64_t ldb,
              double *C, int64_t ldc,
              void *stream);

/*
 * Same operation with HOST buffers (pageable or pinned; pinned buffers let the copies overlap the
 * arithmetic). A and C are streamed through device scratch memory in blocks of 1024 rows (upload,
 * dgemm_f64, download on three streams). B follows the first blocks (three on a large problem) in
 * panels of 1024 rows, and those blocks are multiplied K panel by K panel as the panels arrive,
 * so the arithmetic starts long before B is complete. For those blocks the products of the panels
 * are summed one after the other and the caller's C, which crosses the link behind B, is added
 * last (the sum over k is rounded in that order; one rounding against C, as everywhere). Only the M x N
 * logical part of each row is meaningful; padding columns of the host C are preserved.
 * Synchronous: returns after the result is in the host buffer. Device scratch comes from a memory
 * pool the library owns (stream-ordered allocation) and goes back to it before returning; the
 * pool keeps up to 1.5 GiB mapped between calls, because mapping a gigabyte anew on every call
 * cost more than the copies and the arithmetic of an 8192^3 problem together. The call runs on
 * streams of its own and leases its scratch like any other call, so it may overlap with other
 * calls of this library. Same argument rules and error codes as dgemm_f64 (Section 2.1; the paper's driver
 * likewise owns A, B, C in host memory).
 */
DGEMM_API int dgemm_f64_host(int64_t M, int64_t N, int64_t K,
                   const double *A, int64_t lda,
                   const double *B, int64_t ldb,
                   double *C, int64_t ldc);

/*
 * General form  C = alpha * op(A) * op(B) + beta * C  with op(X) = X or X^T, row-major, FP64,
 * DEVICE pointers. The paper names the scalars and the transposed / strided operand layouts as
 * expressible but leaves them out of its study (Section 2.15, "Other questions": it assumes
 * alpha = beta = 1 and untransposed operands); this entry point is
 * that extension, built on the same kernels as dgemm_f64.
 *
 *   transa  DGEMM_OP_N: A is M x K with lda >= max(1,K).  DGEMM_OP_T: A is stored K x M
 *           (lda >= max(1,M)) and used as its transpose.
 *   transb  DGEMM_OP_N: B is K x N with ldb >= max(1,N).  DGEMM_OP_T: B is stored N x K
 *           (ldb >= max(1,K)) and used as its transpose.
 *   alpha, beta  passed by value. beta == 0: C is an output only, its old contents (NaN or Inf
 *           included) are never read. alpha == 0 or K == 0: A and B are never read and the call
 *           reduces to C = beta * C.
 *
 * Arithmetic: each C element receives beta*C_old + alpha*s, s the K-term inner product summed as
 * in dgemm_f64; alpha = beta = 1 with no transposition gives bit-identical results to dgemm_f64.
 * A transposed operand that is 16-byte aligned with an even leading dimension is used where it
 * lies: the kernels stage the transposed tiles themselves (no extra pass, no extra launch;
 * measured from 512^3 up and on skinny problems: B^T level with the untransposed product, A^T
 * within 0.6 %, 2 % at 512^3). Otherwise (operands that cannot be addressed in place, a very
 * large A^T) a transposed operand is first transposed into device
 * scratch memory owned by the library (an O(MK) or O(KN) pass before O(MNK) arithmetic; the buffer
 * is kept and reused, and leased per call like the rest of the scratch: see dgemm_f64).
 * Same pointer, alignment, aliasing and error rules as dgemm_f64; an op code other than the two
 * above returns DGEMM_ERR_BAD_DIM.
 */
#define DGEMM_OP_N 0
#define DGEMM_OP_T 1
DGEMM_API int dgemm_f64_ex(int transa, int transb, int64_t M, int64_t N, int64_t K,
                           double alpha, const double *A, int64_t lda,
                           const double *B, int64_t ldb,
                           double beta, double *C, int64_t ldc,
                           void *stream);

/*
 * (No counterpart in the paper: an addition for callers that cannot allocate.)
 *
 * C += A*B like dgemm_f64, with K split over several thread blocks and the partial tiles kept in
 * a fixed array that is part of the library image (16 MiB of device memory on every GPU that
 * loads the library, held until the process exits). The call allocates nothing: no cudaMalloc,
 * no cudaFree, no stream-ordered or library allocator. It is meant for callers that are not
 * allowed to allocate at the time of the call, for example because they hold a lock the allocator
 * may need, because they run under a fixed memory budget or inside a latency-critical loop, or
 * because another component owns the device memory pool. dgemm_f64 itself allocates its
 * split-K workspace on first need and so is not suitable for them on small problems.
 *
 * Arguments and error codes are those of dgemm_f64, plus:
 *   split_k   number of K partitions. It is clamped to the number of 16-wide k-blocks, and
 *             partitions that would be empty are dropped. 0 lets the library choose: the most
 *             partitions that the SMs and the array can take (at least 2), or, for a problem
 *             with more than 64 output tiles, 1.
 * Capacity: the array is used only when more than one partition results, and then
 * ceil(M/128) * ceil(N/128) * partitions <= 128 partial tiles must hold. A request beyond that
 * returns DGEMM_ERR_SIZE and launches nothing (use dgemm_f64, or a smaller split_k). A call that
 * ends up with one partition (split_k == 1, the library's choice on a large problem, or
 * K <= 16) runs unsplit, does not touch the array and has no size limit. A negative split_k
 * returns DGEMM_ERR_VARIANT.
 *
 * The first call on each device looks up the array's device address and configures the
 * kernels (no allocation, but several runtime set-up calls): make that first call before any
 * stream capture begins, with the device current. All calls on a device share the
 * one array. Its contents are left over from the previous call; nothing needs clearing because
 * each call overwrites every slot it later reads. Two calls that overlap on the GPU (different
 * streams without ordering between them) race on the array and give undefined results:
 * serialise them, e.g. by using one stream.
 */
DGEMM_API int dgemm_f64_static_ws(int64_t M, int64_t N, int64_t K,
                                  const double *A, int64_t lda,
                                  const double *B, int64_t ldb,
                                  double *C, int64_t ldc,
                                  int split_k, void *stream);

/* Human-readable text for a status code; never NULL; static storage. No counterpart in the paper. */
DGEMM_API const char *dgemm_strerror(int status);

/* Library version as major*10000 + minor*100 + patch. No counterpart in the paper. */
DGEMM_API int dgemm_version(void);

/*
 * Force one kernel variant for subsequent calls of this process (ablation and tests; the
 * paper's analogue is re-running with other pass flags, Section 2.10), or DGEMM_VARIANT_AUTO.
 * Returns DGEMM_OK or DGEMM_ERR_VARIANT. A forced variant that cannot run given operands
 * (DGEMM_VARIANT_TMA on unaligned ones) makes dgemm_f64 return DGEMM_ERR_VARIANT.
 */
DGEMM_API int dgemm_set_variant(int variant);

/* Force a split-K factor (>= 1) for the pipelined variants, or 0 for the built-in heuristic (tests and
 * ablation). No counterpart in the paper: its single core has no use for a K split. */
DGEMM_API int dgemm_set_split_k(int split_k);

/*
 * Testing aid: switches off optional accelerations of the pipelined variants so that tests can
 * exercise the slower code paths and the timing they produce (the operation and its results do
 * not change). Bit flags, 0 restores the default. No counterpart in the paper.
 */
enum {
  DGEMM_TEST_NO_C_PREFETCH = 1, /* do not ask L2 for the C tile ahead of the epilogue           */
  DGEMM_TEST_NO_BLOCKED_B = 2,  /* stage B with eight 2-D copies per stage instead of one 3-D copy */
  DGEMM_TEST_TALL_TILES = 4,    /* 128-row tiles, one CTA per SM, instead of 64-row tiles, two per SM */
  DGEMM_TEST_SMALL_WARP_TILES = 8, /* 32 x 32 warp tiles (twice the warps) instead of 64 x 32           */
  DGEMM_TEST_NO_PACKING = 16,   /* never pack unaligned operands: always use the generic staging      */
  DGEMM_TEST_WS_TWO_CTAS = 32,  /* DGEMM_VARIANT_TMA_WS: 64-row tiles, two CTAs per SM, at any K (the
                                   library itself uses that form only for K < 256)                 */
  DGEMM_TEST_NO_CLUSTER = 128,  /* DGEMM_VARIANT_AUTO never picks the cluster split-K kernel: problems
                                   below one wave of tiles cut K through the workspace instead   */
  DGEMM_TEST_DROP_LOADS = 256   /* failure injection on the host's say-so: the kernels' producers skip their
                                   copies (like a message that is dropped), so the bounded waits of the
                                   arithmetic run out, the kernels report DGEMM_ERR_TIMEOUT through the
                                   status word and return in the ordinary way; C is then unspecified.
                                   Nothing faults, traps or spins without a limit. Use together with
                                   dgemm_set_test_wait_limit, or every wait takes its full four seconds */
};
DGEMM_API int dgemm_set_test_flags(int flags);

/*
 * Testing aid (no counterpart in the paper): the limit of the kernels' main-loop waits in
 * microseconds for subsequent calls, 1 .. 4 000 000, or 0 for the default of four seconds. The
 * separate wait that lets copies in flight land before an aborting thread block exits keeps its
 * own four seconds. Returns DGEMM_OK or DGEMM_ERR_VARIANT.
 */
DGEMM_API int dgemm_set_test_wait_limit(int limit_us);

/*
 * What dgemm_f64 would do with an M x N x K problem under the current variant / split-K / test-flag
 * settings, without touching a device (host logic only; usable on a machine without a GPU):
 * the kernel and tile the library's heuristics choose and how the work is cut (Section 2.10 of
 * the paper explores the same kind of choice by hand). `tma_addressable`: non-zero if A, B and C are
 * 16-byte aligned with even leading dimensions (A and B: or will be after the packing pass) and
 * beta is 0 or 1. `sm_count`:
 * streaming multiprocessors to plan for, 0 = 148 (B200); two CTAs per SM are assumed to fit.
 * Writes 12 ints to `out`: resolved variant, tile rows, tile columns, warp-tile rows, CTAs per
 * SM, grid size, k-blocks (ceil(K/16)), uniform K split, k-blocks per split, tiles run whole,
 * tiles of the last partial wave, k-blocks per CTA span of that wave (== k-blocks: not split).
 * Returns DGEMM_OK, DGEMM_ERR_NULL, DGEMM_ERR_BAD_DIM (a dimension <= 0 or too large) or
 * DGEMM_ERR_VARIANT (the forced variant cannot run such operands).
 */
DGEMM_API int dgemm_plan(int64_t M, int64_t N, int64_t K, int tma_addressable, int sm_count, int *out);

/*
 * Synchronises `stream`, then reads and clears the current device's status word. Returns
 * DGEMM_OK if no kernel reported a problem since the last call, DGEMM_ERR_TIMEOUT if a bounded
 * wait inside a kernel ran out (the kernel then stopped early and C is unspecified), or
 * DGEMM_ERR_CUDA if the synchronisation itself failed. No counterpart in the paper.
 */
DGEMM_API int dgemm_last_device_status(void *stream);

/*
 * Gives the device memory the library holds on the current device back to the system: every
 * scratch lease (an 80 MiB split-K workspace and a packing buffer of up to 2.5 GiB each, as large
 * as the largest packed problem so far; up to four leases) and what the memory pool of
 * dgemm_f64_host keeps mapped (up to 1.5 GiB).
 * All of it comes back on demand. Synchronises the device first (a kernel of an earlier call may
 * still be using the memory), so it must not be called while a stream is being captured. Returns
 * DGEMM_OK, DGEMM_ERR_DEVICE or DGEMM_ERR_CUDA. No counterpart in the paper.
 */
DGEMM_API int dgemm_release_scratch(void);

/*
 * Number of kernels this library has launched so far in this process (all entry points).
 * Monotonic; used by the benchmark to report launches per step. No counterpart in the paper.
 */
DGEMM_API int64_t dgemm_launch_count(void);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper). Launches one thread
 * block that waits on a barrier nobody signals, with a limit of `limit_us` microseconds
 * (clamped to 1 .. 1 000 000). Synchronous. Returns DGEMM_OK if every thread gave up its wait and
 * the kernel returned normally; the device status word then holds DGEMM_ERR_TIMEOUT, which the
 * next dgemm_last_device_status call returns and clears. Nothing traps or hangs.
 */
DGEMM_API int dgemm_selftest_wait_timeout(int limit_us);

/*
 * Measures the FP64 issue rate of the current device with a register-only loop of dependent
 * mma.sync m16n8k8 f64 instructions on all SMs for about `millis` milliseconds (the roofline
 * denominator; the paper computes its machine peak from unit counts in Section 1.2 and this is
 * the measured counterpart). Writes the fused multiply-adds per clock per SM to *fma_per_clk_sm
 * and the sustained rate in TFLOP/s to *tflops (either may be NULL). Synchronous.
 */
DGEMM_API int dgemm_fp64_peak_probe(int millis, double *fma_per_clk_sm, double *tflops);

/*
 * The same measurement for plain FP64 fused multiply-add instructions (16 independent chains per
 * thread, 512 threads per SM): the ceiling of the DGEMM_VARIANT_*_DFMA micro-kernel, next to the
 * tensor-core figure above (the two machine peaks one would compute from unit counts as in
 * Section 1.2; on B200 they differ). Same arguments and return codes.
 */
DGEMM_API int dgemm_fp64_fma_probe(int millis, double *fma_per_clk_sm, double *tflops);

#ifdef __cplusplus
}
#endif
#endif /* DGEMM_H */
