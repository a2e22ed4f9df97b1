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
// One persistent CTA per SM: 8 consumer warps (2 x 4 grid of 64 x 32 warp tiles) and a
// producer warpgroup that hands most of its registers to the consumers (setmaxnreg). Stages are handed over with mbarriers: full[s] (producer -> consumers) and
// empty[s] (consumers -> producer). Every wait is bounded; on expiry the kernel records
// DGEMM_ERR_TIMEOUT in the device status word, drains its own copies and returns.
#pragma once

#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "ptx.cuh"

namespace dgemm {

constexpr int BM = 128;           // CTA tile rows
constexpr int BN = 128;           // CTA tile columns
constexpr int BK = 16;            // k extent of one stage (16 doubles = one 128-byte swizzle row)
constexpr int STAGES = 6;         // pipeline depth
constexpr int CONSUMER_WARPS = 8;
constexpr int PRODUCER_WARPS = 4;  // one warpgroup; it gives most of its registers to the consumers
constexpr int THREADS = (CONSUMER_WARPS + PRODUCER_WARPS) * 32;
constexpr int CONSUMER_REGS = 232;  // 256*232 + 128*40 <= 65536
constexpr int PRODUCER_REGS = 40;
constexpr int A_STAGE_BYTES = BM * BK * 8;  // 16 KiB: 128 rows of 128 bytes
constexpr int B_STAGE_BYTES = BK * BN * 8;  // 16 KiB: 8 boxes of [16 k][16 n] doubles
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int B_BOX_BYTES = BK * 16 * 8;    // 2 KiB
constexpr int SMEM_ALIGN = 1024;            // swizzle pattern repeats every 1024 bytes
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SMEM_ALIGN + 256;
constexpr int STATUS_TIMEOUT = -8;          // DGEMM_ERR_TIMEOUT

struct GemmParams {
  int M, N, K;
  int tiles_m, tiles_n;
  int split_k;            // number of K partitions (>= 1)
  int kblocks_per_split;  // k-blocks (of BK) per partition
  int group_m;            // raster group height in tiles
  const double* A;
  const double* B;
  double* C;
  double* partial;        // split_k > 1: [split][tile][BM*BN] partial sums, else unused
  long long lda, ldb, ldc;
  unsigned long long wait_limit_ns;
  int* status;            // device status word
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

__device__ __forceinline__ void unit_to_tile(const GemmParams& p, int unit, int& tm, int& tn, int& ks) {
  const int tile = unit / p.split_k;
  ks = unit - tile * p.split_k;
  const int per_group = p.group_m * p.tiles_n;
  const int group = tile / per_group;
  const int first_m = group * p.group_m;
  const int gsize = min(p.group_m, p.tiles_m - first_m);
  const int in_group = tile - group * per_group;
  tm = first_m + in_group % gsize;
  tn = in_group / gsize;
}

// Bounded mbarrier wait. Returns false if the CTA is aborting (this or another thread timed out).
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag,
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

template <bool USE_TMA>
__global__ void __launch_bounds__(THREADS, 1)
dgemm_dmma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // tiles at a 1024-byte boundary, barriers behind them
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * STAGE_BYTES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES);
  const uint32_t tiles_u32 = raw + pad;
  const uint32_t full_bar = tiles_u32 + STAGES * STAGE_BYTES;  // full[s]  at full_bar + 8*s
  const uint32_t empty_bar = full_bar + 8 * STAGES;            // empty[s] at empty_bar + 8*s

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar + 8 * s, USE_TMA ? 1 : PRODUCER_WARPS * 32);
      ptx::mbar_init(empty_bar + 8 * s, CONSUMER_WARPS);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
  }
  __syncthreads();

  const int num_units = p.tiles_m * p.tiles_n * p.split_k;
  const int kblocks_total = (p.K + BK - 1) / BK;

  if (warp >= CONSUMER_WARPS) {
    // ------------------------------------------------------------- producer warpgroup
    ptx::setmaxnreg_dec<PRODUCER_REGS>();
    const int pw = warp - CONSUMER_WARPS;  // 0..3
    uint32_t it = 0;  // running stage counter, in lock step with the consumers
    bool ok = true;
    if (USE_TMA) {
      if (pw == 0 && lane == 0) {
        ptx::prefetch_tensormap(&map_a);
        ptx::prefetch_tensormap(&map_b);
        for (int unit = blockIdx.x; unit < num_units && ok; unit += gridDim.x) {
          int tm, tn, ks;
          unit_to_tile(p, unit, tm, tn, ks);
          const int kb0 = ks * p.kblocks_per_split;
          const int kb1 = min(kb0 + p.kblocks_per_split, kblocks_total);
          for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % STAGES;
            const uint32_t ph = (it / STAGES) & 1u;
            if (!wait_bounded(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) { ok = false; break; }
            const uint32_t fb = full_bar + 8 * s;
            const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
            const uint32_t sb = sa + A_STAGE_BYTES;
            ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
            ptx::tma_load_2d(sa, &map_a, kb * BK, tm * BM, fb);
#pragma unroll
            for (int nb = 0; nb < BN / 16; ++nb)
              ptx::tma_load_2d(sb + nb * B_BOX_BYTES, &map_b, tn * BN + nb * 16, kb * BK, fb);
          }
        }
        if (!ok) {
          // aborting: let every copy this thread armed land before the CTA's memory is released
          const uint32_t n_inflight = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
          for (uint32_t q = it - n_inflight; q < it; ++q) {
            const uint32_t s = q % STAGES, ph = (q / STAGES) & 1u;
            const unsigned long long t0 = ptx::globaltimer_ns();
            while (!ptx::mbar_try_wait(full_bar + 8 * s, ph)) {
              if (ptx::globaltimer_ns() - t0 > p.wait_limit_ns) break;
            }
          }
        }
      }
    } else {
      // 8-byte asynchronous copies with zero fill outside the matrices; works for any alignment
      // and any leading dimension. Producer warp pw copies rows 32pw..32pw+31 of the A tile
      // (lanes 0-15 one row's 16 k values, lanes 16-31 the next row's) and columns
      // 32pw..32pw+31 of the B tile (one k row per instruction).
      const int a_r = lane >> 4, a_k = lane & 15;
      for (int unit = blockIdx.x; unit < num_units && ok; unit += gridDim.x) {
        int tm, tn, ks;
        unit_to_tile(p, unit, tm, tn, ks);
        const int kb0 = ks * p.kblocks_per_split;
        const int kb1 = min(kb0 + p.kblocks_per_split, kblocks_total);
        const int m0 = tm * BM, n0 = tn * BN;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!wait_bounded(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) { ok = false; break; }
          const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
          const uint32_t sb = sa + A_STAGE_BYTES;
          const int k0 = kb * BK;
          {
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
          ptx::cp_async_mbar_arrive_noinc(full_bar + 8 * s);
        }
      }
      ptx::cp_async_wait_all();  // nothing of this thread's is in flight when it leaves
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  ptx::setmaxnreg_inc<CONSUMER_REGS>();
  const int g = lane >> 2;   // MMA group id (row of A / column of B fragment)
  const int t = lane & 3;    // thread in group (k index of the fragments)
  const int wm = warp >> 2;  // 0..1 : 64-row slab of the CTA tile
  const int wn = warp & 3;   // 0..3 : 32-column slab
  const int rm = rowmap(g);

  // Byte offsets of this lane's fragments inside a stage, for the two k8 halves h of a stage.
  // A: lane reads k = 8h+2t, 8h+2t+1 of row 64wm + 16mt + {0,8} + rm  (mt adds 2048, +8 rows adds 1024)
  // B: lane reads columns 32wn + 16np + 2g, +1 of k row 8h + 2t + b     (np adds one box)
  uint32_t a_off[2], b_off[2][2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    a_off[h] = (64 * wm + rm) * 128 + (((4 * h + t) ^ rm) << 4);
#pragma unroll
    for (int b = 0; b < 2; ++b)
      b_off[h][b] = A_STAGE_BYTES + (2 * wn) * B_BOX_BYTES + (8 * h + 2 * t + b) * 128 + ((g ^ (2 * t + b)) << 4);
  }

  double acc[4][4][4];  // [mt][nt = 2*np + j][c0..c3]
  uint32_t it = 0;
  bool ok = true;

  for (int unit = blockIdx.x; unit < num_units && ok; unit += gridDim.x) {
    int tm, tn, ks;
    unit_to_tile(p, unit, tm, tn, ks);
    const int kb0 = ks * p.kblocks_per_split;
    const int kb1 = min(kb0 + p.kblocks_per_split, kblocks_total);

#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0;

    for (int kb = kb0; kb < kb1; ++kb, ++it) {
      const uint32_t s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1u;
      if (!wait_bounded(full_bar + 8 * s, ph, abort_flag, p)) { ok = false; break; }
      const uint8_t* st = tiles + s * STAGE_BYTES;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        double2 alo[4], ahi[4], bf[2][2];
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
          alo[mt] = *reinterpret_cast<const double2*>(st + a_off[h] + mt * 2048);
          ahi[mt] = *reinterpret_cast<const double2*>(st + a_off[h] + mt * 2048 + 1024);
        }
#pragma unroll
        for (int np = 0; np < 2; ++np)
#pragma unroll
          for (int b = 0; b < 2; ++b)
            bf[np][b] = *reinterpret_cast<const double2*>(st + b_off[h][b] + np * B_BOX_BYTES);
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int np = 0; np < 2; ++np) {
            ptx::dmma_m16n8k8(acc[mt][2 * np + 0], alo[mt].x, ahi[mt].x, alo[mt].y, ahi[mt].y, bf[np][0].x, bf[np][1].x);
            ptx::dmma_m16n8k8(acc[mt][2 * np + 1], alo[mt].x, ahi[mt].x, alo[mt].y, ahi[mt].y, bf[np][0].y, bf[np][1].y);
          }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty_bar + 8 * s);
    }
    if (!ok) break;

    // ---- epilogue: this lane owns, for each mt, half (rows +0 / +8) and np, four consecutive
    // columns n = 32wn + 16np + 4t + {0,1,2,3} = {nt=2np:c0, nt=2np+1:c0, nt=2np:c1, nt=2np+1:c1}
    const int row_base = tm * BM + 64 * wm + rm;
    const int col_base = tn * BN + 32 * wn + 4 * t;
    if (p.split_k > 1) {
      double* dst = p.partial + ((long long)ks * (p.tiles_m * p.tiles_n) + (unit / p.split_k)) * (long long)(BM * BN);
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int np = 0; np < 2; ++np) {
            const int r = 64 * wm + rm + 16 * mt + 8 * half;
            const int c = 32 * wn + 4 * t + 16 * np;
            ptx::stg256(dst + r * BN + c, acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half],
                        acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]);
          }
    } else {
      const bool interior = (tm * BM + BM <= p.M) && (tn * BN + BN <= p.N);
      const bool vec32 = ((reinterpret_cast<uintptr_t>(p.C) & 31) == 0) && ((p.ldc & 3) == 0);
      if (interior && vec32) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            double* crow = p.C + (long long)(row_base + 16 * mt + 8 * half) * p.ldc + col_base;
            double c0[2], c1[2], c2[2], c3[2];
#pragma unroll
            for (int np = 0; np < 2; ++np) ptx::ldg256(crow + 16 * np, c0[np], c1[np], c2[np], c3[np]);
#pragma unroll
            for (int np = 0; np < 2; ++np)
              ptx::stg256(crow + 16 * np, c0[np] + acc[mt][2 * np][2 * half], c1[np] + acc[mt][2 * np + 1][2 * half],
                          c2[np] + acc[mt][2 * np][2 * half + 1], c3[np] + acc[mt][2 * np + 1][2 * half + 1]);
          }
      } else {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int row = row_base + 16 * mt + 8 * half;
            if (row < p.M) {
              double* crow = p.C + (long long)row * p.ldc;
#pragma unroll
              for (int np = 0; np < 2; ++np) {
                const int col = col_base + 16 * np;
                const double v[4] = {acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half],
                                     acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]};
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (col + e < p.N) crow[col + e] += v[e];
              }
            }
          }
      }
    }
  }
}

// Deterministic split-K reduction: C[i][j] += ((p_0 + p_1) + p_2) + ... in split order.
__global__ void dgemm_splitk_reduce_kernel(const GemmParams p) {
  const int tile = blockIdx.x;
  const int per_group = p.group_m * p.tiles_n;
  const int group = tile / per_group;
  const int first_m = group * p.group_m;
  const int gsize = min(p.group_m, p.tiles_m - first_m);
  const int in_group = tile - group * per_group;
  const int tm = first_m + in_group % gsize;
  const int tn = in_group / gsize;
  const long long num_tiles = (long long)p.tiles_m * p.tiles_n;
  for (int e = threadIdx.x; e < BM * BN; e += blockDim.x) {
    const int r = e / BN, c = e - r * BN;
    const int row = tm * BM + r, col = tn * BN + c;
    if (row < p.M && col < p.N) {
      double sum = p.partial[(long long)tile * (BM * BN) + e];
      for (int s = 1; s < p.split_k; ++s) sum += p.partial[((long long)s * num_tiles + tile) * (BM * BN) + e];
      p.C[(long long)row * p.ldc + col] += sum;
    }
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
