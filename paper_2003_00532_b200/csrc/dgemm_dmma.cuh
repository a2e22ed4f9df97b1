// Pipelined FP64 tensor-core GEMM kernel for sm_100a: C += A*B, row-major.
//
// Mapping of the paper's recipe (Sections 2.4-2.9) onto the GPU:
//   cache tile  (M_C x K_C block of A, K_C x N panel of B)  ->  CTA tile 128 x 128 x 16 per stage
//   packing     (copy into contiguous, conflict-free buffers) ->  asynchronous staging of the
//               A and B block tiles into swizzled shared memory, STAGES deep (this also is the
//               prefetching the paper lists as missing, Section 2.14)
//   register tile M_R x N_R + unroll-and-jam + scalar replacement -> a 64 x 32 accumulator
//               tile per warp held in registers for the whole K loop; C is touched only in
//               the epilogue
//   vectorisation -> mma.sync m16n8k8 f64 (DMMA) and 16-byte shared-memory fragment loads
//   N_C loop the paper left out (Section 2.10) -> grouped tile raster for L2 reuse
//
// Two kernels share the layouts and the epilogue:
//   dgemm_dmma_ws_kernel  warp-specialised: 8 (or 4) consumer warps with 64 x 32 warp tiles and a
//               producer warpgroup that walks the work items and issues the copies; setmaxnreg
//               moves registers from the producers to the consumers; the consumers' k loop is
//               software pipelined. 128 x 128 tiles with one CTA per SM, or 64 x 128 with two.
//   dgemm_dmma_kernel     no producer warp: the load stream runs LOOKAHEAD k-blocks ahead of the
//               arithmetic and across tile boundaries, issued by the warps in turn (TMA) or copied
//               by all threads (8-byte asynchronous copies, any alignment). 64 x 128 tiles with two
//               CTAs per SM, 128 x 128 with one, 256 x 32 for narrow N.
// Persistent CTAs; stages are handed over with mbarriers: full[s] (copies landed) and empty[s]
// (all warps done reading, released behind a proxy fence). Every wait is bounded; on expiry the
// kernel records DGEMM_ERR_TIMEOUT in the device status word, lets its own copies land and
// returns.
#pragma once

#include <type_traits>

#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace dgemm {

constexpr int BM = 128;           // CTA tile rows
constexpr int BN = 128;           // CTA tile columns
constexpr int BK = 16;            // k extent of one stage (16 doubles = one 128-byte swizzle row)
constexpr int STAGES = 6;         // pipeline depth
constexpr int LOOKAHEAD = STAGES - 2;  // k-blocks in flight ahead of the arithmetic
constexpr int WARPS = 8;          // 2 x 4 grid of 64 x 32 warp tiles
constexpr int THREADS = WARPS * 32;
constexpr int A_STAGE_BYTES = BM * BK * 8;  // 16 KiB: 128 rows of 128 bytes
constexpr int B_STAGE_BYTES = BK * BN * 8;  // 16 KiB: 8 boxes of [16 k][16 n] doubles
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int B_BOX_BYTES = BK * 16 * 8;    // 2 KiB
constexpr int SMEM_ALIGN = 1024;            // swizzle pattern repeats every 1024 bytes
// Per-warp staging buffer of the epilogue for C tiles that cannot be accessed 32 bytes at a time
// (edge tiles, C not 32-byte aligned): 8 rows of 32 doubles, 16 bytes of padding per row.
constexpr int EPI_STRIDE = 32 * 8 + 16;
constexpr int EPI_WARP_BYTES = 8 * EPI_STRIDE;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SMEM_ALIGN + 1024 + WARPS * EPI_WARP_BYTES;  // + barriers, abort flag, work-item words, epilogue staging
constexpr int STATUS_TIMEOUT = -8;          // DGEMM_ERR_TIMEOUT
// After an abort a CTA lets the copies it has in flight land before it gives up its shared memory: that
// wait has a limit of its own, not the (possibly shortened) limit of the main-loop waits.
constexpr unsigned long long DRAIN_LIMIT_NS = 4000000000ull;
constexpr int C_PREFETCH_KBLOCKS = 8;       // C tile is requested into L2 this many k-blocks before the tile ends

// Work decomposition. Phase 1: the first `dp_tiles` tiles (in raster order), each split into
// `split_k` equal K partitions, dealt round-robin to the CTAs. Phase 2 (the "tail", the tiles
// that do not fill a whole wave of CTAs): the remaining `tail_tiles` tiles form one long list of
// tail_tiles * kblocks k-block iterations that is cut into equal spans of `tail_ipc` iterations,
// one span per CTA. A span covers the end of one tile and/or the beginning of the next
// (tail_ipc <= kblocks), i.e. at most two segments per CTA. Segments that do not cover a whole
// tile store their partial sums in the workspace and a second kernel adds them to C in a fixed
// order; no CTA ever waits for another one.
struct GemmParams {
  int M, N, K;
  int bm;                 // rows of a CTA tile: 128 (one CTA per SM), 64 (two CTAs per SM) or 256 (narrow tile)
  int bn;                 // columns of a CTA tile: 128, or 32 for the narrow tile
  int tiles_m, tiles_n;
  int kblocks;            // ceil(K / BK)
  int dp_tiles;           // tiles handled in phase 1
  int split_k;            // phase 1: number of K partitions per tile (>= 1)
  int kblocks_per_split;  // phase 1: k-blocks per partition
  int tail_tiles;         // tiles handled in phase 2
  int tail_ipc;           // phase 2: k-block iterations per CTA (1 <= tail_ipc <= kblocks)
  int tail_slot_base;     // first workspace slot of the phase-2 partial tiles
  int group_m;            // raster group height in tiles
  int c_prefetch;         // request the C tile into L2 a few k-blocks before its epilogue
  int b_blocked_map;      // map_b is the 3-D view (16 columns, K, N/16): one copy stages the whole B tile
  int a_blocked_map;      // kernels that stage a transposed A: map_a is the 3-D view (16 rows of op(A), K, M/16)
  int load_c;             // 0: beta == 0, the old C is never read (it may hold NaN)
  double alpha, beta;     // C = beta * C + alpha * (A B); 1, 1 for the paper's C += A B
  const double* A;
  const double* B;
  double* C;
  double* partial;        // workspace: slots of BM*BN doubles; phase 1: slot = ks*dp_tiles + tile
  long long lda, ldb, ldc;
  unsigned long long wait_limit_ns;
  int* status;            // device status word
  int drop_loads;         // testing aid: the producers skip their copies, so that the consumers' waits run out
};

struct Work {
  int tm, tn;    // tile coordinates
  int kb0, kb1;  // k-block range [kb0, kb1)
  int slot;      // workspace slot for the partial tile, or -1: add straight into C
};

// Shared-memory layout of the operand tiles (what the consumer reads and both producers write):
//   A tile: row r (0..127) holds k = 0..15 in 128 bytes; the 16-byte chunk c of row r is stored at
//           chunk position c ^ (r & 7)   (the 128-byte TMA swizzle).
//   B tile: box nb (0..7) holds columns 16*nb..16*nb+15; inside a box row kk (0..15) holds those
//           16 columns in 128 bytes with the same chunk swizzle c ^ (kk & 7).
__device__ __forceinline__ uint32_t a_smem_offset(int r, int kk) {
  return r * 128 + ((((kk >> 1) ^ (r & 7)) << 4) | ((kk & 1) << 3));
}
__device__ __forceinline__ uint32_t b_smem_offset(int kk, int nn) {
  return (nn >> 4) * B_BOX_BYTES + kk * 128 + ((((((nn & 15) >> 1)) ^ (kk & 7)) << 4) | ((nn & 1) << 3));
}

// Row permutation inside a group of 8 tile rows: MMA row index g reads tile row rowmap(g). It
// makes the two rows that share a quarter-warp differ in bit 2, so that one 16-byte fragment
// load per lane touches all 32 banks exactly once.
__device__ __forceinline__ int rowmap(int g) { return ((g & 1) << 2) | (g >> 1); }

// Raster order: groups of `group_m` tile rows, column-major inside a group, so that tiles that run
// at the same time share A row panels and B column panels in L2.
__device__ __forceinline__ void tile_to_mn(const GemmParams& p, int tile, int& tm, int& tn) {
  const int per_group = p.group_m * p.tiles_n;
  const int group = tile / per_group;
  const int first_m = group * p.group_m;
  const int gsize = min(p.group_m, p.tiles_m - first_m);
  const int in_group = tile - group * per_group;
  tm = first_m + in_group % gsize;
  tn = in_group / gsize;
}

// The idx-th work item of CTA `cta` (of `nctas`). Producer and consumers enumerate the same list.
__device__ __forceinline__ bool get_work(const GemmParams& p, int cta, int nctas, int idx, Work& w) {
  const int dp_units = p.dp_tiles * p.split_k;
  const int n1 = cta < dp_units ? (dp_units - cta + nctas - 1) / nctas : 0;
  int tile;
  if (idx < n1) {
    const int unit = cta + idx * nctas;
    tile = unit / p.split_k;
    const int ks = unit - tile * p.split_k;
    w.kb0 = ks * p.kblocks_per_split;
    w.kb1 = min(w.kb0 + p.kblocks_per_split, p.kblocks);
    w.slot = p.split_k > 1 ? ks * p.dp_tiles + tile : -1;
  } else {
    const int j = idx - n1;
    if (j > 1 || p.tail_tiles == 0) return false;
    // 32-bit arithmetic only (the host guarantees tail_tiles * kblocks < 2^31): a 64-bit division
    // would be a called subroutine, which must not run inside the producers' reduced register budget
    const int total = p.tail_tiles * p.kblocks;
    const int start = cta * p.tail_ipc;
    const int end = min(start + p.tail_ipc, total);
    if (start >= end) return false;
    int trel = start / p.kblocks;
    int s0 = start, s1 = min(end, (trel + 1) * p.kblocks);
    if (j == 1) {
      if (s1 >= end) return false;
      s0 = s1;
      s1 = end;
      ++trel;
    }
    tile = p.dp_tiles + trel;
    w.kb0 = s0 - trel * p.kblocks;
    w.kb1 = s1 - trel * p.kblocks;
    w.slot = (w.kb0 == 0 && w.kb1 == p.kblocks) ? -1 : p.tail_slot_base + 2 * cta + j;
  }
  tile_to_mn(p, tile, w.tm, w.tn);
  return true;
}

// ---- rare paths, kept out of line so that the hot k-loop stays small (with two warps per
// scheduler, instruction fetch stalls in a large loop body cost several percent). They take and
// return scalars only; work items travel through a few words of shared memory.

// Work item `idx` of this CTA, written as {tm, tn, kb0, kb1, slot, valid} to shared memory.
__device__ __forceinline__ void fetch_work_inline(const GemmParams& p, int cta, int nctas, int idx, volatile int* out) {
  Work w;
  const bool valid = get_work(p, cta, nctas, idx, w);
  out[0] = w.tm;
  out[1] = w.tn;
  out[2] = w.kb0;
  out[3] = w.kb1;
  out[4] = w.slot;
  out[5] = valid ? 1 : 0;
}
__device__ __noinline__ void fetch_work(const GemmParams& p, int cta, int nctas, int idx, volatile int* out) {
  fetch_work_inline(p, cta, nctas, idx, out);
}

// Asks L2 for rows r0, r0 + rstep, ... of the C tile (tm, tn) ahead of its epilogue.
__device__ __forceinline__ void prefetch_c_rows_inline(const double* C, long long ldc, int M, int N, int bm, int bn,
                                                       int tm, int tn, int r0, int rstep) {
  const int cols = min(bn, N - tn * bn);
  if (cols <= 0) return;
  for (int r = r0; r < bm; r += rstep) {
    const int row = tm * bm + r;
    if (row < M) {
      // one request per 128-byte line of the row segment (measured better than one bulk request per row)
      const double* base = C + (long long)row * ldc + (long long)tn * bn;
      for (int c = 0; c < cols; c += 16) ptx::prefetch_l2(base + c);
      ptx::prefetch_l2(base + cols - 1);
    }
  }
}
__device__ __noinline__ void prefetch_c_rows(const double* C, long long ldc, int M, int N, int bm, int bn, int tm,
                                             int tn, int r0, int rstep) {
  prefetch_c_rows_inline(C, ldc, M, N, bm, bn, tm, tn, r0, rstep);
}

// B stage as eight 2-D boxes of 16 columns (used when N is not a multiple of 16).
__device__ __forceinline__ void tma_load_b_boxes_inline(uint32_t sb, const CUtensorMap* map_b, int n0, int k0,
                                                        uint32_t fb, int boxes = BN / 16) {
  for (int nb = 0; nb < boxes; ++nb) ptx::tma_load_2d(sb + nb * B_BOX_BYTES, map_b, n0 + nb * 16, k0, fb);
}
__device__ __noinline__ void tma_load_b_boxes(uint32_t sb, const CUtensorMap* map_b, int n0, int k0, uint32_t fb,
                                              int boxes) {
  tma_load_b_boxes_inline(sb, map_b, n0, k0, fb, boxes);
}

// A stage of a transposed A (stored K x M): TBM / 16 boxes of [16 k][16 rows of op(A)], as one 3-D copy
// when M is a multiple of 16, else box by box.
__device__ __forceinline__ void tma_load_at(uint32_t sa, const CUtensorMap* map_a, int blocked, int m0, int k0, uint32_t fb,
                                            int boxes) {
  if (blocked) {
    ptx::tma_load_3d(sa, map_a, 0, k0, m0 / 16, fb);
  } else {
    for (int nb = 0; nb < boxes; ++nb) ptx::tma_load_2d(sa + nb * B_BOX_BYTES, map_a, m0 + nb * 16, k0, fb);
  }
}

// Slow part of a bounded mbarrier wait: poll until the phase completes, the CTA aborts, or the
// time limit expires (then record DGEMM_ERR_TIMEOUT and raise the abort flag).
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                       unsigned long long limit_ns, int* status, bool suspend) {
  const unsigned long long t0 = ptx::globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (suspend ? ptx::mbar_try_wait(bar, parity) : ptx::mbar_test_wait(bar, parity)) return true;
    if ((it & 31u) == 0u) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > limit_ns) {
        *abort_flag = 1;
        atomicExch(status, STATUS_TIMEOUT);
        return false;
      }
    }
  }
}

// Fully inlined bounded wait (no call in the caller's hot loop; used where registers are scarce).
__device__ __forceinline__ bool wait_bounded_inline(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                    const GemmParams& p) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = ptx::globaltimer_ns();
  for (uint32_t it = 1;; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 31u) == 0u) {
      if (*abort_flag) return false;
      if (ptx::globaltimer_ns() - t0 > p.wait_limit_ns) {
        *abort_flag = 1;
        atomicExch(p.status, STATUS_TIMEOUT);
        return false;
      }
    }
  }
}

// Bounded mbarrier wait. Returns false if the CTA is aborting (this or another thread timed out).
// SUSPEND = true polls with try_wait (the thread may be suspended for a short, hardware-defined
// time when the phase is not complete: right for the arithmetic waiting for data); SUSPEND = false
// polls with test_wait (never suspends: right for a thread that issues loads in passing).
template <bool SUSPEND = true>
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                             const GemmParams& p) {
  if (SUSPEND ? ptx::mbar_try_wait(bar, parity) : ptx::mbar_test_wait(bar, parity)) return true;
  return wait_slow(bar, parity, abort_flag, p.wait_limit_ns, p.status, SUSPEND);
}

// Position of a lane in the 2 x 4 grid of 64 x 32 warp tiles, and the byte offsets of its fragments
// inside a stage for the two k8 halves h of a stage:
//   A: lane reads k = 8h+2t, 8h+2t+1 of row 64wm + 16mt + {0,8} + rm  (mt adds 2048, +8 rows adds 1024)
//   B: lane reads columns 32wn + 16np + 2g, +1 of k row 8h + 2t + b     (np adds one box)
struct LaneMap {
  int g, t, wm, wn, rm;
  int row0;  // first row of this warp's tile inside the CTA tile (wt_rows * wm)
  uint32_t a_off[2], b_off[2][2];
  uint32_t at_off[2][2];  // transposed A in the stage: [k parity b][rows +0 / +8]
};

//   B stored transposed (`bt`: the stage holds B^T, row n = 128 bytes of 16 k, swizzled like an A tile):
//      lane reads k = 8h+2t, 8h+2t+1 of column 32wn + 16np + 2g + b (np adds 16 rows = 2048 bytes, the
//      size of a box, so the same constant serves); the loaded pair is (k, k+1) of one column instead of
//      (column, column+1) of one k, which only changes the registers a load fills (load_b_pair below).
//   A stored transposed (`at`: the stage holds the K x M matrix's tile as boxes of [16 k][16 rows of
//      op(A)], 128-byte rows, swizzled, exactly the layout of an untransposed B tile): the two k of a
//      fragment pair lie in different 128-byte rows, so a lane reads its four values per 16-row block
//      (rows rm, rm + 8 at k = 8h+2t, 8h+2t+1) with four 8-byte loads instead of two 16-byte ones; the
//      half h only adds 1024 bytes and the 16-row block mt 2048, both immediates.
__device__ __forceinline__ LaneMap make_lane_map(int warp, int lane, int a_stage_bytes = A_STAGE_BYTES, int wt_rows = 64,
                                                 int warps_n = 4, bool bt = false, bool at = false) {
  LaneMap m;
  m.g = lane >> 2;   // MMA group id (row of A / column of B fragment)
  m.t = lane & 3;    // thread in group (k index of the fragments)
  m.wm = warp / warps_n;  // row slab of the CTA tile
  m.wn = warp % warps_n;  // 32-column slab
  m.rm = rowmap(m.g);
  m.row0 = wt_rows * m.wm;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    m.a_off[h] = (m.row0 + m.rm) * 128 + (((4 * h + m.t) ^ m.rm) << 4);
#pragma unroll
    for (int b = 0; b < 2; ++b) {
      m.at_off[h][b] = 0;
      m.b_off[h][b] = bt ? a_stage_bytes + (32 * m.wn + 2 * m.g + b) * 128 + (((4 * h + m.t) ^ ((2 * m.g + b) & 7)) << 4)
                         : a_stage_bytes + (2 * m.wn) * B_BOX_BYTES + (8 * h + 2 * m.t + b) * 128 + ((m.g ^ (2 * m.t + b)) << 4);
    }
  }
  if (at) {
#pragma unroll
    for (int b = 0; b < 2; ++b)
#pragma unroll
      for (int half = 0; half < 2; ++half)
        m.at_off[b][half] = (m.row0 / 16) * B_BOX_BYTES + (2 * m.t + b) * 128 + ((((m.rm >> 1) + 4 * half) ^ (2 * m.t + b)) << 4) + (m.rm & 1) * 8;
  }
  return m;
}

// The arithmetic of one k-block (16 k values) on one stage: acc += A_tile * B_tile for this warp's
// 64 x 32 tile.
template <bool M16 = false, int MT = 4, bool BT = false, bool AT = false>
__device__ __forceinline__ void compute_kblock(const uint8_t* st, const LaneMap& m, double (&acc)[MT][4][4]) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    double2 alo[MT], ahi[MT], bf[2][2];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      if constexpr (AT) {
        alo[mt].x = *reinterpret_cast<const double*>(st + m.at_off[0][0] + h * 1024 + mt * B_BOX_BYTES);
        alo[mt].y = *reinterpret_cast<const double*>(st + m.at_off[1][0] + h * 1024 + mt * B_BOX_BYTES);
        ahi[mt].x = *reinterpret_cast<const double*>(st + m.at_off[0][1] + h * 1024 + mt * B_BOX_BYTES);
        ahi[mt].y = *reinterpret_cast<const double*>(st + m.at_off[1][1] + h * 1024 + mt * B_BOX_BYTES);
      } else {
        alo[mt] = *reinterpret_cast<const double2*>(st + m.a_off[h] + mt * 2048);
        ahi[mt] = *reinterpret_cast<const double2*>(st + m.a_off[h] + mt * 2048 + 1024);
      }
    }
#pragma unroll
    for (int np = 0; np < 2; ++np)
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        const double2 v = *reinterpret_cast<const double2*>(st + m.b_off[h][b] + np * B_BOX_BYTES);
        if constexpr (BT) {  // (k, k+1) of column 2g + b: the x (b = 0) or y (b = 1) halves of both k rows
          if (b == 0) { bf[np][0].x = v.x; bf[np][1].x = v.y; } else { bf[np][0].y = v.x; bf[np][1].y = v.y; }
        } else {
          bf[np][b] = v;
        }
      }
    // Eight k values per block as two k4 steps (x: k = 8h + 2t, y: k = 8h + 2t + 1) of the
    // m8n8k4 shape; rows g (alo) and g + 8 (ahi) are separate 8 x 8 tiles.
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int np = 0; np < 2; ++np) {
        if (M16) {  // same arithmetic with the 16 x 8 x 8 shape: a quarter of the instructions
          ptx::dmma_m16n8k8(acc[mt][2 * np + 0], alo[mt].x, ahi[mt].x, alo[mt].y, ahi[mt].y, bf[np][0].x, bf[np][1].x);
          ptx::dmma_m16n8k8(acc[mt][2 * np + 1], alo[mt].x, ahi[mt].x, alo[mt].y, ahi[mt].y, bf[np][0].y, bf[np][1].y);
          continue;
        }
        ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], alo[mt].x, bf[np][0].x);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], ahi[mt].x, bf[np][0].x);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], alo[mt].x, bf[np][0].y);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], ahi[mt].x, bf[np][0].y);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], alo[mt].y, bf[np][1].x);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], ahi[mt].y, bf[np][1].x);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], alo[mt].y, bf[np][1].y);
        ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], ahi[mt].y, bf[np][1].y);
      }
  }
}

// The micro-kernel swap (the paper's "outer MLIR, inner BLIS" experiment, Section 2.12, turned
// around: same staging, pipeline, raster and epilogue, another inner kernel). Plain FP64 FMAs on a
// register tile instead of tensor-core MMAs: every lane keeps the very 8 x 8 scattered elements of
// the warp tile that the MMA layout gives it (rows row0 + rm + 8i, columns 32wn + 16np + 4t + e),
// so the epilogue is shared unchanged. Per k a lane needs 8 values of A (one per owned row) and 8
// of B (one per owned column) for 64 FMAs; they come as 16-byte loads of two consecutive k (A) and
// two consecutive columns (B) from the same swizzled stage layout. Lanes with equal g read the
// same A words and lanes with equal t the same B words (broadcast), and the 8 rows / 4 column
// chunks of a load fall into distinct banks. k runs in ascending order inside the k-block.
template <int MT = 4>
__device__ __forceinline__ void compute_kblock_dfma(const uint8_t* st, const LaneMap& m, int a_stage_bytes,
                                                    double (&acc)[MT][4][4]) {
  const uint8_t* a_base = st + (m.row0 + m.rm) * 128;
  const uint8_t* b_base = st + a_stage_bytes + (2 * m.wn) * B_BOX_BYTES;
#pragma unroll
  for (int kp = 0; kp < BK / 2; ++kp) {
    double2 a[MT][2];  // [16-row block][rows +0 / +8]: k = 2kp (x), 2kp + 1 (y)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int half = 0; half < 2; ++half)
        a[mt][half] = *reinterpret_cast<const double2*>(a_base + (16 * mt + 8 * half) * 128 + ((kp ^ m.rm) << 4));
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
      const int k = 2 * kp + kk;
      double2 b[2][2];  // [np][q]: columns 16np + 4t + 2q (x), + 1 (y)
#pragma unroll
      for (int np = 0; np < 2; ++np)
#pragma unroll
        for (int q = 0; q < 2; ++q)
          b[np][q] = *reinterpret_cast<const double2*>(b_base + np * B_BOX_BYTES + k * 128 + (((2 * m.t + q) ^ (k & 7)) << 4));
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const double av = kk == 0 ? a[mt][half].x : a[mt][half].y;
#pragma unroll
          for (int np = 0; np < 2; ++np)
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              // column offset e = 2q (x), 2q + 1 (y) lives in acc[mt][2np + (e & 1)][2 half + (e >> 1)]
              acc[mt][2 * np + 0][2 * half + q] = fma(av, b[np][q].x, acc[mt][2 * np + 0][2 * half + q]);
              acc[mt][2 * np + 1][2 * half + q] = fma(av, b[np][q].y, acc[mt][2 * np + 1][2 * half + q]);
            }
        }
    }
  }
}

// ---- the same arithmetic in software-pipelined pieces ---------------------------------------------
// One half k-block (8 k values) of fragments for a warp tile of 16*MT rows x 32 columns: 48
// registers for MT = 4. The warp-specialised kernel keeps two of them, so that the loads of the next half
// (and, across a k-block boundary, the barrier test before them) are issued ahead of the MMAs of
// the current half and a warp can feed the FP64 pipe without a gap at the boundary.
template <int MT>
struct Frags {
  double2 alo[MT], ahi[MT], bf[2][2];
};

// The A fragments of 16-row block MT_ for the k8 half H, rows +0 (lo) or +8 (hi): one 16-byte load from
// an untransposed A tile, two 8-byte loads from a transposed one (same registers either way).
template <int H, int MT_, bool HI, bool AT, int MT>
__device__ __forceinline__ void load_a_pair(Frags<MT>& f, uint32_t stage, const LaneMap& m) {
  double2& dst = HI ? f.ahi[MT_] : f.alo[MT_];
  if constexpr (!AT) {
    ptx::lds128_off<MT_ * 2048 + (HI ? 1024 : 0)>(stage + m.a_off[H], dst.x, dst.y);
  } else {
    ptx::lds64_off<MT_ * B_BOX_BYTES + H * 1024>(stage + m.at_off[0][HI ? 1 : 0], dst.x);
    ptx::lds64_off<MT_ * B_BOX_BYTES + H * 1024>(stage + m.at_off[1][HI ? 1 : 0], dst.y);
  }
}

template <int I, int N, typename F>
__device__ __forceinline__ void static_for(F&& f) {
  if constexpr (I < N) {
    f(std::integral_constant<int, I>());
    static_for<I + 1, N>(f);
  }
}

// `stage` is the shared-memory address of the stage; H selects k = 8H .. 8H+7.
// One 16-byte B fragment load: with B as stored (BT = false) the pair is columns 2g, 2g+1 of k row b;
// with B^T in the stage it is k rows 0, 1 of column 2g + b. Same address arithmetic, other registers.
template <int NP, int B, bool BT, int MT>
__device__ __forceinline__ void load_b_pair(Frags<MT>& f, uint32_t addr) {
  if constexpr (!BT) ptx::lds128_off<NP * B_BOX_BYTES>(addr, f.bf[NP][B].x, f.bf[NP][B].y);
  else if constexpr (B == 0) ptx::lds128_off<NP * B_BOX_BYTES>(addr, f.bf[NP][0].x, f.bf[NP][1].x);
  else ptx::lds128_off<NP * B_BOX_BYTES>(addr, f.bf[NP][0].y, f.bf[NP][1].y);
}

template <int H, int MT, bool BT = false, bool AT = false>
__device__ __forceinline__ void load_frags(Frags<MT>& f, uint32_t stage, const LaneMap& m) {
  static_for<0, MT>([&](auto mt) {
    load_a_pair<H, mt.value, false, AT>(f, stage, m);
    load_a_pair<H, mt.value, true, AT>(f, stage, m);
  });
  static_for<0, 2>([&](auto np) {
    load_b_pair<np.value, 0, BT>(f, stage + m.b_off[H][0]);
    load_b_pair<np.value, 1, BT>(f, stage + m.b_off[H][1]);
  });
}

// The MMAs of row blocks [MT0, MT1) of one half k-block.
template <int MT0, int MT1, int MT>
__device__ __forceinline__ void mma_frags(double (&acc)[MT][4][4], const Frags<MT>& f) {
#pragma unroll
  for (int mt = MT0; mt < MT1; ++mt)
#pragma unroll
    for (int np = 0; np < 2; ++np) {
      ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], f.alo[mt].x, f.bf[np][0].x);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], f.ahi[mt].x, f.bf[np][0].x);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], f.alo[mt].x, f.bf[np][0].y);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], f.ahi[mt].x, f.bf[np][0].y);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], f.alo[mt].y, f.bf[np][1].x);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], f.ahi[mt].y, f.bf[np][1].x);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], f.alo[mt].y, f.bf[np][1].y);
      ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], f.ahi[mt].y, f.bf[np][1].y);
    }
}

// One of the 12 fragment loads of a half k-block, numbered so that the ones needed first by the
// MMAs come first: 0..3 = B (np, b), then per row block alo, ahi.
template <int H, int I, bool BT, bool AT, int MT>
__device__ __forceinline__ void load_frag_piece(Frags<MT>& f, uint32_t stage, const LaneMap& m) {
  if constexpr (I < 4) {
    constexpr int np = I >> 1, b = I & 1;
    load_b_pair<np, b, BT>(f, stage + m.b_off[H][b]);
  } else if constexpr (I < 4 + 2 * MT) {
    constexpr int mt = (I - 4) >> 1;
    load_a_pair<H, mt, ((I - 4) & 1) != 0, AT>(f, stage, m);
  }
}

// The MMAs of row blocks [MT0, MT1) of the half k-block in `cur`, with the loads [L0, L1) of half
// HN (into `nxt`, from `stage_n`) spread between them, so that the loads neither arrive in a burst
// nor wait behind the arithmetic.
template <int MT0, int MT1, int HN, int L0, int L1, bool BT = false, bool AT = false, int MT = 4>
__device__ __forceinline__ void mma_frags_loading(double (&acc)[MT][4][4], const Frags<MT>& cur, Frags<MT>& nxt,
                                                  uint32_t stage_n, const LaneMap& m) {
  constexpr int GROUPS = 2 * (MT1 - MT0);
  static_for<0, GROUPS>([&](auto gi) {
    constexpr int g = gi.value;
    constexpr int mt = MT0 + g / 2, np = g % 2;
    // loads [lo, hi) of this group: an even share of L1 - L0
    constexpr int lo = L0 + (L1 - L0) * g / GROUPS, hi = L0 + (L1 - L0) * (g + 1) / GROUPS;
    static_for<lo, hi>([&](auto li) { load_frag_piece<HN, li.value, BT, AT>(nxt, stage_n, m); });
    ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], cur.alo[mt].x, cur.bf[np][0].x);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], cur.ahi[mt].x, cur.bf[np][0].x);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], cur.alo[mt].x, cur.bf[np][0].y);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], cur.ahi[mt].x, cur.bf[np][0].y);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 0][0], acc[mt][2 * np + 0][1], cur.alo[mt].y, cur.bf[np][1].x);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 0][2], acc[mt][2 * np + 0][3], cur.ahi[mt].y, cur.bf[np][1].x);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 1][0], acc[mt][2 * np + 1][1], cur.alo[mt].y, cur.bf[np][1].y);
    ptx::dmma_m8n8k4(acc[mt][2 * np + 1][2], acc[mt][2 * np + 1][3], cur.ahi[mt].y, cur.bf[np][1].y);
  });
}

// Releases a stage: one arrival per warp on its `empty` mbarrier, after which the producer may
// refill it with TMA copies. Those copies write through the asynchronous proxy while the fragment
// loads above read through the generic proxy, and an mbarrier arrive alone does not order the two:
// without the proxy fence the refill could overwrite rows that a fragment load had yet to read
// (observed as sporadically wrong 8-row blocks, most often on K = 64 tiles; reproduced by
// tests/test_gpu_stress.py with a plain arrive). Every lane fences its own loads, the warp
// synchronises, lane 0 arrives.
__device__ __forceinline__ void release_stage(uint32_t empty_bar_s, int lane) {
  ptx::fence_proxy_async();
  __syncwarp();
  if (lane == 0) ptx::mbar_arrive(empty_bar_s);
}

// Epilogue of one work item: adds the accumulators to the C tile (or stores them as a partial tile
// in the workspace when the item covers only part of K).
template <int MT_PER_BATCH, int MT = 4, bool STAGED = false>
__device__ __forceinline__ void store_tile(const GemmParams& p, const Work& w, const LaneMap& m, double (&acc)[MT][4][4],
                                           uint32_t epi_buf = 0) {
  const int tm = w.tm, tn = w.tn;
  // This lane owns, for each mt, half (rows +0 / +8) and np, four consecutive
  // columns n = 32wn + 16np + 4t + {0,1,2,3} = {nt=2np:c0, nt=2np+1:c0, nt=2np:c1, nt=2np+1:c1}
  const int row_base = tm * p.bm + m.row0 + m.rm;
  const int col_base = tn * p.bn + 32 * m.wn + 4 * m.t;
  if (w.slot >= 0) {
    double* dst = p.partial + (long long)w.slot * (long long)(BM * BN);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int half = 0; half < 2; ++half)
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          const int r = m.row0 + m.rm + 16 * mt + 8 * half;
          const int c = 32 * m.wn + 4 * m.t + 16 * np;
          ptx::stg256(dst + r * p.bn + c, acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half],
                      acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]);
        }
  } else {
    if (p.alpha != 1.0) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[mt][nt][e] *= p.alpha;
    }
    const bool interior = (tm * p.bm + p.bm <= p.M) && (tn * p.bn + p.bn <= p.N);
    const bool vec32 = ((reinterpret_cast<uintptr_t>(p.C) & 31) == 0) && ((p.ldc & 3) == 0);
    if (interior && vec32) {
      // batches of 4 * MT_PER_BATCH outstanding 32-byte loads per thread, then the adds and stores
#pragma unroll
      for (int mp = 0; mp < MT / MT_PER_BATCH; ++mp) {
        double cin[MT_PER_BATCH][2][2][4];
        if (p.load_c) {
#pragma unroll
          for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const double* crow = p.C + (long long)(row_base + 16 * (MT_PER_BATCH * mp + mq) + 8 * half) * p.ldc + col_base;
#pragma unroll
              for (int np = 0; np < 2; ++np)
                ptx::ldg256(crow + 16 * np, cin[mq][half][np][0], cin[mq][half][np][1], cin[mq][half][np][2],
                            cin[mq][half][np][3]);
            }
        } else {
#pragma unroll
          for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
            for (int half = 0; half < 2; ++half)
#pragma unroll
              for (int np = 0; np < 2; ++np)
#pragma unroll
                for (int e = 0; e < 4; ++e) cin[mq][half][np][e] = -0.0;  // fma(-0, beta, x) == x for every x, -0 included
        }
#pragma unroll
        for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int mt = MT_PER_BATCH * mp + mq;
            double* crow = p.C + (long long)(row_base + 16 * mt + 8 * half) * p.ldc + col_base;
#pragma unroll
            for (int np = 0; np < 2; ++np)
              // beta == 1: fma(c, 1, acc) rounds once, exactly like c + acc
              ptx::stg256(crow + 16 * np, fma(cin[mq][half][np][0], p.beta, acc[mt][2 * np][2 * half]),
                          fma(cin[mq][half][np][1], p.beta, acc[mt][2 * np + 1][2 * half]),
                          fma(cin[mq][half][np][2], p.beta, acc[mt][2 * np][2 * half + 1]),
                          fma(cin[mq][half][np][3], p.beta, acc[mt][2 * np + 1][2 * half + 1]));
          }
      }
    } else if constexpr (STAGED) {
      // Edge tiles and C that is not 32-byte aligned, through this warp's staging buffer: 8 rows of
      // the warp tile at a time go to shared memory in row-major order and come back with lane L
      // holding column L, so that every global access of the warp is one 256-byte row segment
      // (8 or 9 sectors) instead of 32 scattered 8-byte pieces (32 sectors, a quarter of each
      // used: 4096 x 4096 x 64 with ldc = 4098 ran 125 us that way against 89 us with ldc = 4096).
      const int lane = 4 * m.g + m.t;
      const int col = tn * p.bn + 32 * m.wn + lane;
      const bool col_in = col < p.N;
      const uint32_t wr = epi_buf + m.rm * EPI_STRIDE + m.t * 32;  // this lane's 4 columns of row rm (np adds 128 bytes)
      const uint32_t rd = epi_buf + lane * 8;                     // column `lane` of row j at + j * EPI_STRIDE
      // Per batch of MT_PER_BATCH 16-row blocks: all old C values are requested first (as many bytes
      // in flight per warp as on the 32-byte path), the accumulators go through the buffer while
      // those loads are under way, and every store comes after every load of the batch (a load
      // behind a store would have to wait for it: they may alias as far as the compiler knows).
#pragma unroll
      for (int mp = 0; mp < MT / MT_PER_BATCH; ++mp) {
        double cin[MT_PER_BATCH][2][8];
        const int row0 = tm * p.bm + m.row0 + 16 * MT_PER_BATCH * mp;
        double* cbase = p.C + (long long)row0 * p.ldc + col;
#pragma unroll
        for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
          for (int half = 0; half < 2; ++half)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int r = 16 * mq + 8 * half + j;
              cin[mq][half][j] = (p.load_c && col_in && row0 + r < p.M) ? cbase[(long long)r * p.ldc] : -0.0;
            }
#pragma unroll
        for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int mt = MT_PER_BATCH * mp + mq;
#pragma unroll
            for (int np = 0; np < 2; ++np) {
              ptx::sts128(wr + np * 128, acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half]);
              ptx::sts128(wr + np * 128 + 16, acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]);
            }
            __syncwarp();
            double v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = ptx::lds64_f64(rd + j * EPI_STRIDE);
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int r = 16 * mq + 8 * half + j;
              if (col_in && row0 + r < p.M) cbase[(long long)r * p.ldc] = fma(cin[mq][half][j], p.beta, v[j]);
            }
          }
      }
    } else {
      // Edge tiles and C that is not 32-byte aligned: 8-byte accesses with a bounds check per
      // element, in the same batches as above. All loads of a batch are issued before the first
      // store: interleaved, every load would have to wait for the store before it (they may alias
      // as far as the compiler knows) and the epilogue would run at one memory latency per element
      // (a 3192 x 125 x 32 problem took 31 us that way, 10 us with the batches).
#pragma unroll
      for (int mp = 0; mp < MT / MT_PER_BATCH; ++mp) {
        double cin[MT_PER_BATCH][2][2][4];
#pragma unroll
        for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int row = row_base + 16 * (MT_PER_BATCH * mp + mq) + 8 * half;
            const double* crow = p.C + (long long)row * p.ldc;
#pragma unroll
            for (int np = 0; np < 2; ++np)
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int col = col_base + 16 * np + e;
                cin[mq][half][np][e] = (p.load_c && row < p.M && col < p.N) ? crow[col] : -0.0;
              }
          }
#pragma unroll
        for (int mq = 0; mq < MT_PER_BATCH; ++mq)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int mt = MT_PER_BATCH * mp + mq;
            const int row = row_base + 16 * mt + 8 * half;
            if (row >= p.M) continue;
            double* crow = p.C + (long long)row * p.ldc;
#pragma unroll
            for (int np = 0; np < 2; ++np) {
              const int col = col_base + 16 * np;
              const double v[4] = {acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half],
                                   acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]};
#pragma unroll
              for (int e = 0; e < 4; ++e)
                if (col + e < p.N) crow[col + e] = fma(cin[mq][half][np][e], p.beta, v[e]);
            }
          }
      }
    }
  }
}

// Adds `count` partial tiles (workspace slots slot_of(0..count-1), in that order) to elements
// [e_begin, e_end) of the C tile (tm, tn): C = beta*C + alpha*(((p_0 + p_1) + p_2) + ...).
// Deterministic. The partial tiles were written by other CTAs, possibly of this same kernel, so
// they are read past L1.
template <int U, typename SlotFn>
__device__ __forceinline__ void reduce_range(const GemmParams& p, int tm, int tn, int count, SlotFn slot_of, int e_begin,
                                             int e_end, int tid, int nthreads) {
  // U element pairs per thread and pass, all loads of a segment issued before any is used: the
  // reads come from L2 with a latency of hundreds of cycles, so their number in flight is what
  // counts (U = 1 for the reduction kernels, whose many CTAs provide it)
  for (int e0 = e_begin + 2 * tid; e0 < e_end; e0 += 2 * nthreads * U) {
    double2 sum[U];
    const double* src = p.partial + (long long)slot_of(0) * (BM * BN);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int e = e0 + 2 * nthreads * u;
      sum[u] = e < e_end ? __ldcg(reinterpret_cast<const double2*>(src + e)) : make_double2(0.0, 0.0);
    }
    int s = 1;
    // eight partial tiles per round trip while there are that many (tiles cut into many pieces)
    for (; s + 8 <= count; s += 8) {
      double2 w[8][U];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const double* sq = p.partial + (long long)slot_of(s + q) * (BM * BN);
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int e = e0 + 2 * nthreads * u;
          w[q][u] = e < e_end ? __ldcg(reinterpret_cast<const double2*>(sq + e)) : make_double2(0.0, 0.0);
        }
      }
#pragma unroll
      for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int u = 0; u < U; ++u) {
          sum[u].x += w[q][u].x;
          sum[u].y += w[q][u].y;
        }
    }
    for (; s < count; ++s) {
      src = p.partial + (long long)slot_of(s) * (BM * BN);
      double2 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int e = e0 + 2 * nthreads * u;
        v[u] = e < e_end ? __ldcg(reinterpret_cast<const double2*>(src + e)) : make_double2(0.0, 0.0);
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        sum[u].x += v[u].x;
        sum[u].y += v[u].y;
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int e = e0 + 2 * nthreads * u;
      if (e >= e_end) continue;
      const int r = e / p.bn, c = e - r * p.bn;
      const int row = tm * p.bm + r, col = tn * p.bn + c;
      if (row < p.M && col < p.N) {
        double* dst = p.C + (long long)row * p.ldc + col;
        const double sx = sum[u].x * p.alpha, sy = sum[u].y * p.alpha;  // exact for alpha == 1
        dst[0] = p.load_c ? fma(dst[0], p.beta, sx) : sx;
        if (col + 1 < p.N) dst[1] = p.load_c ? fma(dst[1], p.beta, sy) : sy;
      }
    }
  }
}

// Shape of the inline kernel for a tile height TBM: 128 rows -> 8 warps, 6 stages of 32 KB, one CTA
// per SM; 64 rows -> 4 warps, 4 stages of 24 KB, two CTAs per SM (they drift out of phase, so one
// CTA's k-block boundaries and epilogues overlap with the other's arithmetic).
template <int TBM, int WTM = 64, int TBN = BN>
struct TileCfg {
  static constexpr int MT_ = WTM / 16;                        // m16 row blocks per warp tile
  static constexpr int WARPS_N = TBN / 32;                    // warp grid: (TBM / WTM) x (TBN / 32)
  static constexpr int WARPS_ = (TBM / WTM) * WARPS_N;
  static constexpr int THREADS_ = WARPS_ * 32;
  static constexpr int CTAS_PER_SM = (TBM == 128 && TBN == 128) ? 1 : 2;
  static constexpr int A_BYTES = TBM * BK * 8;
  static constexpr int B_BYTES = BK * TBN * 8;
  static constexpr int STAGE_BYTES_ = A_BYTES + B_BYTES;
  // as many stages as fit: 6 x 32 KB (one CTA per SM), 4 x 24 KB or 3 x 36 KB (two CTAs per SM)
  static constexpr int STAGES_ = CTAS_PER_SM == 1 ? 6 : (STAGE_BYTES_ <= 24 * 1024 ? 4 : 3);
  static constexpr int LOOKAHEAD_ = STAGES_ > 3 ? STAGES_ - 2 : STAGES_ - 1;
  // epilogue staging where it fits: not next to the three 36 KB stages of the 256 x 32 tile, nor with
  // the 8 or 16 warps of the tiles built from 32 x 32 warp tiles (they keep the scattered 8-byte accesses)
  static constexpr bool EPI_STAGED = !(TBM == 256 || (WTM == 32 && TBM >= 64));
  static constexpr int EPI_OFFSET = STAGES_ * STAGE_BYTES_ + 2048;  // from the first stage
  static constexpr int SMEM_BYTES_ = STAGES_ * STAGE_BYTES_ + SMEM_ALIGN + 2048 + (EPI_STAGED ? WARPS_ * EPI_WARP_BYTES : 0);
};

// MICRO selects the inner kernel: tensor-core MMAs (the product), or plain FMAs on the same register
// tile (the micro-kernel swap of the ablation ladder).
constexpr int MICRO_DMMA = 0;
constexpr int MICRO_DFMA = 1;

// BT: map_b describes B as stored transposed (N x K, the general entry point's op(B) = B^T) and the
// stage holds B^T: no transposing pass in HBM. TMA staging only.
// AT: likewise map_a describes A as stored transposed (K x M) and the stage holds that tile.
template <bool USE_TMA, int TBM, int WTM = 64, int TBN = BN, int MICRO = MICRO_DMMA, bool BT = false, bool AT = false>
__global__ void __launch_bounds__(TileCfg<TBM, WTM, TBN>::THREADS_, TileCfg<TBM, WTM, TBN>::CTAS_PER_SM)
dgemm_dmma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ GemmParams p) {
  constexpr int MT = TileCfg<TBM, WTM, TBN>::MT_;
  constexpr int WARPS_N = TileCfg<TBM, WTM, TBN>::WARPS_N;
  constexpr int STAGES = TileCfg<TBM, WTM, TBN>::STAGES_;
  constexpr int LOOKAHEAD = TileCfg<TBM, WTM, TBN>::LOOKAHEAD_;
  constexpr int WARPS = TileCfg<TBM, WTM, TBN>::WARPS_;
  constexpr int THREADS = TileCfg<TBM, WTM, TBN>::THREADS_;
  constexpr int A_STAGE_BYTES = TileCfg<TBM, WTM, TBN>::A_BYTES;
  constexpr int STAGE_BYTES = TileCfg<TBM, WTM, TBN>::STAGE_BYTES_;
  extern __shared__ uint8_t smem_raw[];
  // tiles at a 1024-byte boundary, barriers behind them
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * STAGE_BYTES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES);
  volatile int* work_words = abort_flag + 8;  // per warp: 8 words for the load cursor's item, 8 for the current item
  const uint32_t tiles_u32 = raw + pad;
  const uint32_t full_bar = tiles_u32 + STAGES * STAGE_BYTES;  // full[s]  at full_bar + 8*s
  const uint32_t empty_bar = full_bar + 8 * STAGES;            // empty[s] at empty_bar + 8*s

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar + 8 * s, USE_TMA ? 1 : THREADS);
      ptx::mbar_init(empty_bar + 8 * s, WARPS);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  ptx::grid_dependency_wait();  // everything above overlaps the tail of the previous kernel in the stream

  const int cta = blockIdx.x, nctas = gridDim.x;
  // Every thread follows the load stream. TMA staging: the k-blocks are issued by the warps in
  // turn (k-block number i by lane 0 of warp i mod 8), which spreads the cost of issuing over the
  // four schedulers. Generic staging: every thread copies its share of each stage.
  if (USE_TMA && tid == 0) {
    ptx::prefetch_tensormap(&map_a);
    ptx::prefetch_tensormap(&map_b);
  }

  // State of the load stream: the k-blocks of this CTA's work items in order, LOOKAHEAD k-blocks
  // ahead of the arithmetic and running across tile boundaries, so that the first stages of the
  // next tile are in flight while the current tile's epilogue runs. Uniform over the CTA.
  volatile int* cur_words = work_words + 16 * warp;
  volatile int* item_words = cur_words + 8;
  int cur_idx = 0, cur_tm, cur_tn, cur_kb, cur_kb1, cur_pf, cur_valid;
  auto cursor_load = [&]() {
    fetch_work(p, cta, nctas, cur_idx, cur_words);
    __syncwarp();
    cur_tm = cur_words[0];
    cur_tn = cur_words[1];
    cur_kb = cur_words[2];
    cur_kb1 = cur_words[3];
    cur_valid = cur_words[5];
    // k-block at which the C tile is requested into L2, or -1 (partial tiles do not read C)
    cur_pf = (cur_words[4] < 0 && p.c_prefetch) ? max(cur_kb, cur_kb1 - C_PREFETCH_KBLOCKS) : -1;
    __syncwarp();
  };
  cursor_load();
  uint32_t lit = 0;  // k-blocks issued so far
  bool ok = true;

  // Issues the next k-block of the load stream into stage lit % STAGES (after that stage's previous
  // contents have been released by all warps). Returns false if the CTA is aborting.
  auto issue_next = [&]() -> bool {
    if (!cur_valid) return true;
    const uint32_t s = lit % STAGES;
    const uint32_t ph = (lit / STAGES) & 1u;
    const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
    const uint32_t sb = sa + A_STAGE_BYTES;
    const uint32_t fb = full_bar + 8 * s;
    const int kb = cur_kb;
    if (USE_TMA) {
      // Only the issuing warp learns at once that its wait gave up; the other warps see the abort
      // flag in their own next wait. (A vote in every warp on every k-block costs 0.5 % at 8192^3.)
      if (warp == (int)(lit % WARPS)) {
        int good = 1;
        if (lane == 0) {
          if (!wait_bounded<false>(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) {
            good = 0;
          } else if (!p.drop_loads) {
            ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
            if constexpr (AT) {
              tma_load_at(sa, &map_a, p.a_blocked_map, cur_tm * TBM, kb * BK, fb, TBM / 16);
            } else {
              ptx::tma_load_2d(sa, &map_a, kb * BK, cur_tm * TBM, fb);
            }
            if constexpr (BT) {
              ptx::tma_load_2d(sb, &map_b, kb * BK, cur_tn * TBN, fb);  // rows n of B^T, 16 k each
            } else if (p.b_blocked_map) {
              ptx::tma_load_3d(sb, &map_b, 0, kb * BK, cur_tn * (TBN / 16), fb);
            } else {
              tma_load_b_boxes(sb, &map_b, cur_tn * TBN, kb * BK, fb, TBN / 16);
            }
          }
        }
        if (!__all_sync(0xffffffffu, good)) return false;
      }
    } else {
      if (!wait_bounded<false>(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) return false;
      if (!p.drop_loads) {
      // 8-byte asynchronous copies with zero fill outside the matrices; any alignment, any leading
      // dimension. A: 16 consecutive threads copy the 16 k values of one row (8 rows per thread);
      // B: 32 consecutive threads copy 32 consecutive columns of one k row (8 k rows per thread).
      const int m0 = cur_tm * TBM, n0 = cur_tn * TBN, k0 = kb * BK;
      // a stage that lies wholly inside the matrices (the common case) skips the bounds logic:
      // the copies are a third of this loader's instructions, the predicates were the rest
      const bool inside = (m0 + TBM <= p.M) && (n0 + TBN <= p.N) && (k0 + BK <= p.K);
      {
        const int a_k = tid & 15, row0 = tid >> 4;
        const int k = k0 + a_k;
        const bool kin = k < p.K;
        const double* src = p.A + (long long)(m0 + row0) * p.lda + k;
        const uint32_t dst_base = sa + ((a_k & 1) << 3);
        constexpr int ROW_STEP = THREADS / 16;
        if (inside) {
#pragma unroll
          for (int i = 0; i < TBM / ROW_STEP; ++i) {
            const int row = row0 + ROW_STEP * i;
            ptx::cp_async_8(dst_base + row * 128 + (((a_k >> 1) ^ (row & 7)) << 4), src + (long long)(ROW_STEP * i) * p.lda, 8u);
          }
        } else {
#pragma unroll
          for (int i = 0; i < TBM / ROW_STEP; ++i) {
            const int row = row0 + ROW_STEP * i;
            const bool in = kin && (m0 + row < p.M);
            const uint32_t dst = dst_base + row * 128 + (((a_k >> 1) ^ (row & 7)) << 4);
            ptx::cp_async_8(dst, in ? (const void*)(src + (long long)(ROW_STEP * i) * p.lda) : (const void*)p.A, in ? 8u : 0u);
          }
        }
      }
      {
        const int nn = tid % TBN, kk0 = tid / TBN;
        const bool nin = n0 + nn < p.N;
        const double* src = p.B + (long long)(k0 + kk0) * p.ldb + (n0 + nn);
        const uint32_t dst_base = sb + (nn >> 4) * B_BOX_BYTES + ((nn & 1) << 3);
        const int chunk = (nn & 15) >> 1;
        constexpr int K_STEP = THREADS / TBN;
        if (inside) {
#pragma unroll
          for (int i = 0; i < BK / K_STEP; ++i) {
            const int kk = kk0 + K_STEP * i;
            ptx::cp_async_8(dst_base + kk * 128 + ((chunk ^ (kk & 7)) << 4), src + (long long)(K_STEP * i) * p.ldb, 8u);
          }
        } else {
#pragma unroll
          for (int i = 0; i < BK / K_STEP; ++i) {
            const int kk = kk0 + K_STEP * i;
            const bool in = nin && (k0 + kk < p.K);
            const uint32_t dst = dst_base + kk * 128 + ((chunk ^ (kk & 7)) << 4);
            ptx::cp_async_8(dst, in ? (const void*)(src + (long long)(K_STEP * i) * p.ldb) : (const void*)p.B, in ? 8u : 0u);
          }
        }
      }
      ptx::cp_async_mbar_arrive_noinc(fb);
      }
    }
    if (kb == cur_pf) {
      // TMA staging: the issuing warp's lanes take 4 rows each; generic: one row per thread of the first 128
      if (USE_TMA) {
        if (warp == (int)(lit % WARPS)) prefetch_c_rows(p.C, p.ldc, p.M, p.N, TBM, TBN, cur_tm, cur_tn, lane, 32);
      } else {
        prefetch_c_rows(p.C, p.ldc, p.M, p.N, TBM, TBN, cur_tm, cur_tn, tid, THREADS);
      }
    }
    ++lit;
    if (++cur_kb >= cur_kb1) {
      ++cur_idx;
      cursor_load();
    }
    return true;
  };

  for (int i = 0; i < LOOKAHEAD && ok; ++i) ok = issue_next();

  static_assert(!(BT || AT) || (USE_TMA && MICRO == MICRO_DMMA), "the transposed stages exist for TMA staging and the MMA micro-kernel");
  const LaneMap lm = make_lane_map(warp, lane, A_STAGE_BYTES, WTM, WARPS_N, BT, AT);

  double acc[MT][4][4];  // [mt][nt = 2*np + j][c0..c3]
  uint32_t it = 0;      // k-blocks consumed so far
  Work w;

  for (int idx = 0; ok; ++idx) {
    fetch_work(p, cta, nctas, idx, item_words);
    __syncwarp();
    w.tm = item_words[0];
    w.tn = item_words[1];
    w.kb0 = item_words[2];
    w.kb1 = item_words[3];
    w.slot = item_words[4];
    const int valid = item_words[5];
    __syncwarp();
    if (!valid) break;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0;

    for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
      const uint32_t s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1u;
      if (!wait_bounded(full_bar + 8 * s, ph, abort_flag, p)) { ok = false; break; }
      if constexpr (MICRO == MICRO_DFMA) compute_kblock_dfma<MT>(tiles + s * STAGE_BYTES, lm, A_STAGE_BYTES, acc);
      else compute_kblock<false, MT, BT, AT>(tiles + s * STAGE_BYTES, lm, acc);
      release_stage(empty_bar + 8 * s, lane);
      // keep the load stream LOOKAHEAD k-blocks ahead: refill the stage released two k-blocks ago
      if (!issue_next()) { ok = false; break; }
    }
    if (!ok) break;

    store_tile<(MT >= 4 ? 2 : 1), MT, TileCfg<TBM, WTM, TBN>::EPI_STAGED>(
        p, w, lm, acc, tiles_u32 + TileCfg<TBM, WTM, TBN>::EPI_OFFSET + warp * EPI_WARP_BYTES);
  }

  // Leaving. After a normal run every copy that was issued has been consumed. After an abort,
  // copies may still be in flight into this CTA's shared memory: let them land first.
  if (!USE_TMA) ptx::cp_async_wait_all();
  if (USE_TMA && !ok && !p.drop_loads && tid == 0) {
    const uint32_t n_inflight = lit < (uint32_t)STAGES ? lit : (uint32_t)STAGES;
    for (uint32_t q = lit - n_inflight; q < lit; ++q) {
      const uint32_t s = q % STAGES, ph = (q / STAGES) & 1u;
      const unsigned long long t0 = ptx::globaltimer_ns();
      while (!ptx::mbar_try_wait(full_bar + 8 * s, ph)) {
        if (ptx::globaltimer_ns() - t0 > DRAIN_LIMIT_NS) break;
      }
    }
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Warp-specialised variant: 8 consumer warps as above plus one producer warpgroup (384 threads).
// The producers hand most of their registers to the consumers (setmaxnreg: 232 / 40; the pool is
// what the CTA owns at launch, 384 x 168, so 256 x 232 + 128 x 40 must not exceed it). The
// producer runs up to STAGES k-blocks ahead. TMA staging: lane 0 of the first producer warp issues
// the copies; generic staging: the four producer warps copy 32 rows of A and 32 columns of B each.
constexpr int WS_EPI_BATCH = 2;  // 16-row blocks of C loaded per batch in the epilogue (8 loads of 32 bytes in flight
                                 // per thread; 4 spills heavily at 232 registers, 1 leaves the load latency exposed:
                                 // rank-k K = 64 1300 us with 1, 1252 us with 2)
constexpr int WS_PRODUCER_WARPS = 4;
constexpr int WS_THREADS = (WARPS + WS_PRODUCER_WARPS) * 32;
constexpr int WS_CONSUMER_REGS = 232;
constexpr int WS_PRODUCER_REGS = 40;

template <int TBM>
struct WsCfg {
  static constexpr int CONSUMER_WARPS = TBM / 16;  // a (TBM / 64) x 4 grid of 64 x 32 warp tiles
  static constexpr int THREADS_ = (CONSUMER_WARPS + WS_PRODUCER_WARPS) * 32;
  static constexpr int CTAS_PER_SM = TBM == 128 ? 1 : 2;
  static constexpr int A_BYTES = TBM * BK * 8;
  static constexpr int STAGE_BYTES_ = A_BYTES + B_STAGE_BYTES;
  static constexpr int STAGES_ = TBM == 128 ? 6 : 4;
  static constexpr int EPI_OFFSET = STAGES_ * STAGE_BYTES_ + 1024;  // epilogue staging, from the first stage
  static constexpr int SMEM_BYTES_ = STAGES_ * STAGE_BYTES_ + SMEM_ALIGN + 2048 + CONSUMER_WARPS * EPI_WARP_BYTES;
  // register pool = THREADS_ x registers at launch (168 or 128): consumers x 232 + 128 x producers
  static constexpr int PRODUCER_REGS = TBM == 128 ? WS_PRODUCER_REGS : 24;
};

template <bool USE_TMA, int TBM = BM, bool BT = false, bool AT = false>
__global__ void __launch_bounds__(WsCfg<TBM>::THREADS_, WsCfg<TBM>::CTAS_PER_SM)
dgemm_dmma_ws_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ GemmParams p) {
  static_assert(USE_TMA || TBM == 128, "generic staging needs the 128-row producer layout and 40 producer registers");
  static_assert(!(BT || AT) || USE_TMA, "the transposed stages exist for TMA staging only");
  constexpr int STAGES = WsCfg<TBM>::STAGES_;
  constexpr int WARPS = WsCfg<TBM>::CONSUMER_WARPS;
  constexpr int A_STAGE_BYTES = WsCfg<TBM>::A_BYTES;
  constexpr int STAGE_BYTES = WsCfg<TBM>::STAGE_BYTES_;
  constexpr int WS_THREADS = WsCfg<TBM>::THREADS_;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * STAGE_BYTES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES);
  volatile int* work_words = abort_flag + 8;  // 8 words per warp (12 warps)
  const uint32_t tiles_u32 = raw + pad;
  const uint32_t full_bar = tiles_u32 + STAGES * STAGE_BYTES;
  const uint32_t empty_bar = full_bar + 8 * STAGES;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar + 8 * s, USE_TMA ? 1 : WS_PRODUCER_WARPS * 32);
      ptx::mbar_init(empty_bar + 8 * s, WARPS);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  ptx::grid_dependency_wait();  // everything above overlaps the tail of the previous kernel in the stream

  const int cta = blockIdx.x, nctas = gridDim.x;
  volatile int* item_words = work_words + 8 * warp;
  Work w;
  uint32_t it = 0;  // running k-block counter, the same sequence in producers and consumers
  bool ok = true;

  if (warp >= WARPS) {
    // ------------------------------------------------------------------ producer warpgroup
    ptx::setmaxnreg_dec<WsCfg<TBM>::PRODUCER_REGS>();
    const int pw = warp - WARPS;
    const bool active = USE_TMA ? (pw == 0) : true;
    if (USE_TMA && pw == 0 && lane == 0) {
      ptx::prefetch_tensormap(&map_a);
      ptx::prefetch_tensormap(&map_b);
    }
    for (int idx = 0; active && ok; ++idx) {
      fetch_work_inline(p, cta, nctas, idx, item_words);
      __syncwarp();
      w.tm = item_words[0];
      w.tn = item_words[1];
      w.kb0 = item_words[2];
      w.kb1 = item_words[3];
      w.slot = item_words[4];
        const int valid = item_words[5];
      __syncwarp();
      if (!valid) break;
      const int kb_pf = (w.slot < 0 && p.c_prefetch) ? max(w.kb0, w.kb1 - C_PREFETCH_KBLOCKS) : -1;
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1u;
        const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
        const uint32_t sb = sa + A_STAGE_BYTES;
        const uint32_t fb = full_bar + 8 * s;
        if (USE_TMA) {
          int good = 1;
          if (lane == 0) {
            if (!wait_bounded_inline(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) {
              good = 0;
            } else if (!p.drop_loads) {
              ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
              if constexpr (AT) {
                tma_load_at(sa, &map_a, p.a_blocked_map, w.tm * TBM, kb * BK, fb, TBM / 16);
              } else {
                ptx::tma_load_2d(sa, &map_a, kb * BK, w.tm * TBM, fb);
              }
              if constexpr (BT) {
                ptx::tma_load_2d(sb, &map_b, kb * BK, w.tn * BN, fb);  // rows n of B^T, 16 k each
              } else if (p.b_blocked_map) {
                ptx::tma_load_3d(sb, &map_b, 0, kb * BK, w.tn * (BN / 16), fb);
              } else {
                tma_load_b_boxes_inline(sb, &map_b, w.tn * BN, kb * BK, fb);
              }
            }
          }
          if (!__all_sync(0xffffffffu, good)) { ok = false; break; }
          if (kb == kb_pf) prefetch_c_rows_inline(p.C, p.ldc, p.M, p.N, TBM, BN, w.tm, w.tn, lane, 32);
        } else {
          if (!wait_bounded_inline(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) { ok = false; break; }
          const int m0 = w.tm * BM, n0 = w.tn * BN, k0 = kb * BK;
          if (!p.drop_loads) {
          {
            const int a_r = lane >> 4, a_k = lane & 15;
            const int k = k0 + a_k;
            const bool kin = k < p.K;
            const int row0 = 32 * pw + a_r;
            const double* src = p.A + (long long)(m0 + row0) * p.lda + k;
            const uint32_t dst_base = sa + ((a_k & 1) << 3);
#pragma unroll 4
            for (int r = 0; r < 32; r += 2) {
              const int row = row0 + r;
              const bool in = kin && (m0 + row < p.M);
              const uint32_t dst = dst_base + row * 128 + (((a_k >> 1) ^ (row & 7)) << 4);
              ptx::cp_async_8(dst, in ? (const void*)(src + (long long)r * p.lda) : (const void*)p.A, in ? 8u : 0u);
            }
          }
          {
            const int nn = 32 * pw + lane;
            const bool nin = n0 + nn < p.N;
            const double* src = p.B + (long long)k0 * p.ldb + (n0 + nn);
            const uint32_t dst_base = sb + (nn >> 4) * B_BOX_BYTES + ((nn & 1) << 3);
            const int chunk = (nn & 15) >> 1;
#pragma unroll 4
            for (int kk = 0; kk < BK; ++kk) {
              const bool in = nin && (k0 + kk < p.K);
              const uint32_t dst = dst_base + kk * 128 + ((chunk ^ (kk & 7)) << 4);
              ptx::cp_async_8(dst, in ? (const void*)(src + (long long)kk * p.ldb) : (const void*)p.B, in ? 8u : 0u);
            }
          }
          ptx::cp_async_mbar_arrive_noinc(fb);
          }
          if (kb == kb_pf) prefetch_c_rows_inline(p.C, p.ldc, p.M, p.N, BM, BN, w.tm, w.tn, 32 * pw + lane, BM);
        }
      }
    }
    if (!USE_TMA) ptx::cp_async_wait_all();
    if (USE_TMA && !ok && !p.drop_loads && pw == 0 && lane == 0) {
      // aborting: let every copy this thread armed land before the CTA's memory is released
      const uint32_t n_inflight = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
      for (uint32_t q = it - n_inflight; q < it; ++q) {
        const uint32_t s = q % STAGES, ph = (q / STAGES) & 1u;
        const unsigned long long t0 = ptx::globaltimer_ns();
        while (!ptx::mbar_try_wait(full_bar + 8 * s, ph)) {
          if (ptx::globaltimer_ns() - t0 > DRAIN_LIMIT_NS) break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ consumer warps
    ptx::setmaxnreg_inc<WS_CONSUMER_REGS>();
    const LaneMap lm = make_lane_map(warp, lane, A_STAGE_BYTES, 64, 4, BT, AT);
    double acc[4][4][4];
    for (int idx = 0; ok && get_work(p, cta, nctas, idx, w); ++idx) {
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0;
      Frags<4> f0, f1;
      {
        const uint32_t s = it % STAGES;
        if (!wait_bounded_inline(full_bar + 8 * s, (it / STAGES) & 1u, abort_flag, p)) { ok = false; break; }
        load_frags<0, 4, BT, AT>(f0, tiles_u32 + s * STAGE_BYTES, lm);
      }
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % STAGES;
        const uint32_t s1 = (it + 1) % STAGES;
        const uint32_t ph1 = ((it + 1) / STAGES) & 1u;
        const bool more = kb + 1 < w.kb1;
        const bool ready = more && ptx::mbar_test_wait(full_bar + 8 * s1, ph1);
        mma_frags_loading<0, 4, 1, 0, 12, BT, AT>(acc, f0, f1, tiles_u32 + s * STAGE_BYTES, lm);
        if (more) {
          if (!ready && !wait_bounded_inline(full_bar + 8 * s1, ph1, abort_flag, p)) { ok = false; break; }
          mma_frags_loading<0, 2, 0, 0, 6, BT, AT>(acc, f1, f0, tiles_u32 + s1 * STAGE_BYTES, lm);
          release_stage(empty_bar + 8 * s, lane);
          mma_frags_loading<2, 4, 0, 6, 12, BT, AT>(acc, f1, f0, tiles_u32 + s1 * STAGE_BYTES, lm);
        } else {
          mma_frags<0, 2>(acc, f1);
          release_stage(empty_bar + 8 * s, lane);
          mma_frags<2, 4>(acc, f1);
        }
      }
      if (!ok) break;
      store_tile<WS_EPI_BATCH, 4, true>(p, w, lm, acc, tiles_u32 + WsCfg<TBM>::EPI_OFFSET + warp * EPI_WARP_BYTES);
    }
  }
  ptx::named_barrier_sync(1, WS_THREADS);  // all warps leave together
}

// Adds `count` partial tiles (workspace slots slot[0..count)) to the C tile (tm, tn) in that order:
// C[i][j] += ((p_0 + p_1) + p_2) + ...  Deterministic. A tile is reduced by REDUCE_CHUNKS CTAs
// (blockIdx.y), each taking BM / REDUCE_CHUNKS consecutive rows.
constexpr int REDUCE_CHUNKS = 16;
constexpr int REDUCE_THREADS = 256;

template <typename SlotFn>
__device__ __forceinline__ void reduce_tile(const GemmParams& p, int tm, int tn, int count, SlotFn slot_of) {
  const int chunk_elems = p.bm * p.bn / REDUCE_CHUNKS;  // a slot holds a bm x bn tile, row-major
  const int e0 = blockIdx.y * chunk_elems;
  reduce_range<1>(p, tm, tn, count, slot_of, e0, e0 + chunk_elems, threadIdx.x, REDUCE_THREADS);
}

// Phase-1 split-K reduction: tile t has its split_k partials in slots ks*dp_tiles + t.
__global__ void dgemm_splitk_reduce_kernel(const GemmParams p) {
  ptx::grid_dependency_wait();
  const int tile = blockIdx.x;
  int tm, tn;
  tile_to_mn(p, tile, tm, tn);
  reduce_tile(p, tm, tn, p.split_k, [&](int s) { return s * p.dp_tiles + tile; });
}

// Phase-2 (tail) reduction: tail tile `trel` was covered by the spans of CTAs c_first..c_last; CTA c
// stored its part in slot tail_slot_base + 2c + j, j = 0 if the span starts inside this tile.
__global__ void dgemm_tail_reduce_kernel(const GemmParams p) {
  ptx::grid_dependency_wait();
  const int trel = blockIdx.x;
  const int lo = trel * p.kblocks, hi = lo + p.kblocks;
  const int c_first = lo / p.tail_ipc;
  const int c_last = (hi - 1) / p.tail_ipc;
  if (c_first == c_last && c_first * p.tail_ipc == lo && p.tail_ipc == p.kblocks) return;  // went straight to C
  int tm, tn;
  tile_to_mn(p, p.dp_tiles + trel, tm, tn);
  reduce_tile(p, tm, tn, c_last - c_first + 1, [&](int s) {
    const int c = c_first + s;
    const int j = (c * p.tail_ipc >= lo) ? 0 : 1;
    return p.tail_slot_base + 2 * c + j;
  });
}

// Packing pass for operands that TMA cannot address (base not 16-byte aligned or odd leading
// dimension): copies a rows x cols matrix into a 16-byte aligned buffer with an even leading
// dimension. This is the paper's packing step (Section 2.6) done once in HBM instead of per block;
// it moves O(n^2) bytes for O(n^3) work. One thread per pair of columns.
// The packing pass for one or two operands in one launch (blockIdx.z selects the operand; blocks
// beyond the smaller operand's extent return at once). Launched with programmatic stream
// serialization: waits for the kernel before it, which may still be reading the scratch it writes.
struct PackOp {
  const double* src;
  long long ld_src;
  int rows, cols;
  double* dst;
  long long ld_dst;
};
__global__ void dgemm_pack2_kernel(const PackOp a, const PackOp b) {
  ptx::grid_dependency_wait();
  const PackOp& o = blockIdx.z == 0 ? a : b;
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= o.cols) return;
  for (int r0 = blockIdx.y * 8; r0 < o.rows; r0 += gridDim.y * 8) {  // gridDim.y may be capped
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = r0 + i;
      if (r < o.rows) {
        const double* s = o.src + (long long)r * o.ld_src + c;
        double2 v;
        v.x = s[0];
        v.y = (c + 1 < o.cols) ? s[1] : 0.0;
        *reinterpret_cast<double2*>(o.dst + (long long)r * o.ld_dst + c) = v;
      }
    }
  }
}

__global__ void dgemm_pack_kernel(const double* __restrict__ src, long long ld_src, int rows, int cols,
                                  double* __restrict__ dst, long long ld_dst) {
  const int c = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (c >= cols) return;
  for (int r0 = blockIdx.y * 8; r0 < rows; r0 += gridDim.y * 8) {  // gridDim.y may be capped
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = r0 + i;
      if (r < rows) {
        const double* s = src + (long long)r * ld_src + c;
        double2 v;
        v.x = s[0];
        v.y = (c + 1 < cols) ? s[1] : 0.0;
        *reinterpret_cast<double2*>(dst + (long long)r * ld_dst + c) = v;
      }
    }
  }
}

// Out-of-place transpose dst[c][r] = src[r][c] of a rows x cols matrix (32 x 32 tiles through
// shared memory, both sides coalesced): turns a transposed operand of the general entry point
// into the row-major layout the tile loaders read. Block (32, 8).
__global__ void dgemm_transpose_kernel(const double* __restrict__ src, long long ld_src, int rows, int cols,
                                       double* __restrict__ dst, long long ld_dst) {
  __shared__ double tile[32][33];
  ptx::grid_dependency_wait();  // launched with programmatic stream serialization, like the packing pass
  const int c0 = blockIdx.x * 32;
  for (int r0 = blockIdx.y * 32; r0 < rows; r0 += gridDim.y * 32) {  // gridDim.y may be capped
#pragma unroll
    for (int i = threadIdx.y; i < 32; i += 8) {
      const int r = r0 + i, c = c0 + threadIdx.x;
      if (r < rows && c < cols) tile[i][threadIdx.x] = src[(long long)r * ld_src + c];
    }
    __syncthreads();
#pragma unroll
    for (int i = threadIdx.y; i < 32; i += 8) {
      const int c = c0 + i, r = r0 + threadIdx.x;
      if (r < rows && c < cols) dst[(long long)c * ld_dst + r] = tile[threadIdx.x][i];
    }
    __syncthreads();
  }
}

// C = beta * C over the logical M x N part (alpha == 0 or K == 0 in the general entry point);
// beta == 0 stores zeros without reading. One thread per element, grid-stride over rows.
__global__ void dgemm_scale_kernel(double* C, long long ldc, int M, int N, double beta) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= N) return;
  for (int i = blockIdx.y; i < M; i += gridDim.y) {
    double* c = C + (long long)i * ldc + j;
    *c = (beta == 0.0) ? 0.0 : *c * beta;
  }
}

// C += T, element by element (both row-major with their own leading dimensions; 16-byte aligned,
// even leading dimensions and an even number of columns): the host entry point adds the caller's C
// to a product that was started before that C had crossed the host link.
__global__ void dgemm_add_kernel(double* C, long long ldc, const double* T, long long ldt, int M, int N) {
  const int j = 2 * (blockIdx.x * blockDim.x + threadIdx.x);
  if (j >= N) return;
  for (int i = blockIdx.y; i < M; i += gridDim.y) {
    double2* c = reinterpret_cast<double2*>(C + (long long)i * ldc + j);
    const double2 t = *reinterpret_cast<const double2*>(T + (long long)i * ldt + j);
    double2 v = *c;
    v.x += t.x;
    v.y += t.y;
    *c = v;
  }
}

// Self-test of the bounded wait: one CTA waits on an mbarrier that nobody signals. The wait gives up
// after p.wait_limit_ns, records DGEMM_ERR_TIMEOUT in the status word and the kernel returns
// normally (nothing traps, nothing spins without a limit).
__global__ void dgemm_wait_timeout_selftest_kernel(const __grid_constant__ GemmParams p, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();
  ptx::grid_dependency_wait();  // everything above overlaps the tail of the previous kernel in the stream
  const bool ok = wait_bounded(ptx::smem_u32(&bar), 0u, &abort_flag, p);
  if (!ok) atomicAdd(gave_up, 1);
}

// Rung 1 of the ladder: tiles of A and B in shared memory, still one C element per thread and no
// register tile (the paper's tiling + packing stage, Sections 2.4-2.6, before unroll-and-jam):
// every FMA needs two shared-memory loads. 32 x 32 threads per CTA, k in steps of 32, plain loads.
constexpr int SMEM_RUNG_TILE = 32;
__global__ void __launch_bounds__(SMEM_RUNG_TILE * SMEM_RUNG_TILE)
dgemm_smem_kernel(int M, int N, int K, const double* __restrict__ A, long long lda, const double* __restrict__ B,
                  long long ldb, double* C, long long ldc) {
  constexpr int T = SMEM_RUNG_TILE;
  __shared__ double As[T][T + 1];
  __shared__ double Bs[T][T];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int j = blockIdx.x * T + tx;
  for (int i0 = blockIdx.y * T; i0 < M; i0 += gridDim.y * T) {  // gridDim.y may be capped
    const int i = i0 + ty;
    double acc = 0.0;
    for (int k0 = 0; k0 < K; k0 += T) {
      As[ty][tx] = (i < M && k0 + tx < K) ? A[(long long)i * lda + k0 + tx] : 0.0;
      Bs[ty][tx] = (k0 + ty < K && j < N) ? B[(long long)(k0 + ty) * ldb + j] : 0.0;
      __syncthreads();
#pragma unroll
      for (int k = 0; k < T; ++k) acc = fma(As[ty][k], Bs[k][tx], acc);
      __syncthreads();
    }
    if (i < M && j < N) C[(long long)i * ldc + j] += acc;
  }
}

// Rung 0 of the ladder: the naive nest with one thread per C element (Section 2.1).
__global__ void dgemm_naive_kernel(int M, int N, int K, const double* __restrict__ A, long long lda,
                                   const double* __restrict__ B, long long ldb, double* C, long long ldc) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int i = blockIdx.y * blockDim.y + threadIdx.y;
  if (i >= M || j >= N) return;
  double acc = 0.0;
  for (int k = 0; k < K; ++k) acc = fma(A[(long long)i * lda + k], B[(long long)k * ldb + j], acc);
  C[(long long)i * ldc + j] += acc;
}

}  // namespace dgemm
