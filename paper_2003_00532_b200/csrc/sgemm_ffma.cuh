// Single-precision C += A*B for sm_100a: exact binary32 arithmetic on the FP32 pipe (FFMA), fed
// by the same TMA + mbarrier staging as the FP64 kernels. The paper's SGEMM (Section 2.13) is its
// DGEMM nest with f64 replaced by f32 and a wider register tile; here the register tile is 8 x 8
// per thread, the CTA tile 128 x 128 x 32, 256 threads, two CTAs per SM.
//
// The FP32 pipe issues one warp-wide FFMA per scheduler per clock (128 FFMA/clk/SM), so the bound
// is instruction issue: per 4 k values a thread issues 256 FFMAs, 8 + 8 16-byte shared-memory
// loads and a few address operations.
#pragma once

#include <cstdint>
#include <cuda.h>

#include "ptx.cuh"

namespace sgemm {

using namespace dgemm::ptx;

#ifndef SGEMM_CTAS
#define SGEMM_CTAS 1
#endif
constexpr int TM = SGEMM_CTAS == 1 ? 256 : 128;  // CTA tile rows
constexpr int RPT = TM / 16;                       // rows per thread
constexpr int TN = 128;  // CTA tile columns
constexpr int TK = 32;   // k extent of a stage: 32 floats = one 128-byte swizzle row
constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int A_BYTES = TM * TK * 4;        // 16 KiB: 128 rows of 128 bytes
constexpr int B_BOX_BYTES = TK * 32 * 4;    // 4 KiB: [32 k][32 columns]
constexpr int B_BYTES = (TN / 32) * B_BOX_BYTES;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int STAGES = SGEMM_CTAS == 1 ? 4 : 3;
constexpr int LOOKAHEAD = 2;                // k-blocks in flight ahead of the arithmetic
constexpr int SMEM_ALIGN = 1024;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SMEM_ALIGN + 256;
constexpr int STATUS_TIMEOUT = -8;          // DGEMM_ERR_TIMEOUT


struct Params {
  int M, N, K;
  int tiles_m, tiles_n;
  int kblocks;         // ceil(K / TK)
  int group_m;         // raster group height in tiles
  int b_blocked_map;   // map_b is the 3-D view (32 columns, K, N/32): one copy stages the whole B tile
  const float* A;
  const float* B;
  float* C;
  long long lda, ldb, ldc;
  unsigned long long wait_limit_ns;
  int* status;
};

// Tiles are numbered in groups of `group_m` tile rows, column-major inside a group, so that the
// tiles running at the same time share A row panels and B column panels in L2.
__device__ __forceinline__ void tile_to_mn(const Params& p, int tile, int& tm, int& tn) {
  const int per_group = p.group_m * p.tiles_n;
  const int g = tile / per_group;
  const int r = tile - g * per_group;
  const int rows = min(p.group_m, p.tiles_m - g * p.group_m);
  tn = r / rows;
  tm = g * p.group_m + (r - tn * rows);
}

// Polls an mbarrier phase; gives up after p.wait_limit_ns, records the timeout and raises the
// CTA's abort flag. Never spins without a limit.
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns,
                                       int* status) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > limit_ns) {
      atomicExch(status, STATUS_TIMEOUT);
      *abort_flag = 1;
      return false;
    }
  }
}

__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort_flag, const Params& p) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, abort_flag, p.wait_limit_ns, p.status);
}

__global__ void __launch_bounds__(THREADS, SGEMM_CTAS)
sgemm_ffma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  const uint32_t tiles_u32 = raw + pad;
  const uint32_t full_bar = tiles_u32 + STAGES * STAGE_BYTES;  // full[s]  at full_bar + 8*s
  const uint32_t empty_bar = full_bar + 8 * STAGES;            // empty[s] at empty_bar + 8*s
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tiles + STAGES * STAGE_BYTES + 16 * STAGES);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar + 8 * s, 1);
      mbar_init(empty_bar + 8 * s, WARPS);
    }
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  __syncthreads();

  const int cta = blockIdx.x, nctas = gridDim.x;
  const int ntiles = p.tiles_m * p.tiles_n;

  // Load stream: the k-blocks of this CTA's tiles (cta, cta + nctas, ...) in order, LOOKAHEAD
  // k-blocks ahead of the arithmetic and across tile boundaries. Every thread follows the cursor;
  // k-block number i is issued by lane 0 of warp i mod 8.
  int l_tile = cta, l_kb = 0, l_tm = 0, l_tn = 0;
  if (l_tile < ntiles) tile_to_mn(p, l_tile, l_tm, l_tn);
  uint32_t lit = 0;
  auto issue_next = [&]() -> bool {
    if (l_tile >= ntiles) return true;
    if (warp == (int)(lit % WARPS)) {
      int good = 1;
      if (lane == 0) {
        const uint32_t s = lit % STAGES;
        const uint32_t ph = (lit / STAGES) & 1u;
        const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
        const uint32_t sb = sa + A_BYTES;
        const uint32_t fb = full_bar + 8 * s;
        if (wait_bounded(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) {
          mbar_arrive_expect_tx(fb, STAGE_BYTES);
          tma_load_2d(sa, &map_a, l_kb * TK, l_tm * TM, fb);
          if (p.b_blocked_map) {
            tma_load_3d(sb, &map_b, 0, l_kb * TK, l_tn * (TN / 32), fb);
          } else {
            for (int nb = 0; nb < TN / 32; ++nb) tma_load_2d(sb + nb * B_BOX_BYTES, &map_b, l_tn * TN + nb * 32, l_kb * TK, fb);
          }
        } else {
          good = 0;
        }
      }
      if (!__all_sync(0xffffffffu, good)) return false;
    }
    ++lit;
    if (++l_kb >= p.kblocks) {
      l_kb = 0;
      l_tile += nctas;
      if (l_tile < ntiles) tile_to_mn(p, l_tile, l_tm, l_tn);
    }
    return true;
  };

  bool ok = true;
  for (int i = 0; i < LOOKAHEAD && ok; ++i) ok = issue_next();

  // Thread (ty, tx) of the 16 x 16 grid owns rows ty + 16 i (i < 8) and columns 4 tx .. 4 tx + 3 and
  // 64 + 4 tx .. 64 + 4 tx + 3. Shared-memory layout (what TMA writes with the 128-byte swizzle):
  //   A: row r holds k = 0..31 in 128 bytes, 16-byte chunk c at position c ^ (r & 7);
  //   B: box nb holds columns 32 nb .. 32 nb + 31; in a box, row k holds them in 128 bytes, chunk
  //      c at position c ^ (k & 7).
  // A fragment load: 4 consecutive k of one row (the 16 tx lanes of a row share the address);
  // B fragment load: 4 consecutive columns of one k (8 lanes cover a 128-byte row).
  const int ty = tid >> 4, tx = tid & 15;
  const uint32_t a_off = (uint32_t)ty * 128u;            // + i * 2048 + ((kg ^ (ty & 7)) << 4)
  const uint32_t a_sw = (uint32_t)(ty & 7);
  const uint32_t b_off = (uint32_t)A_BYTES + (uint32_t)(tx >> 3) * B_BOX_BYTES;  // + k * 128 + (((tx & 7) ^ (k & 7)) << 4)
  const uint32_t b_ch = (uint32_t)(tx & 7);

  float2 acc[RPT][4];  // [row i][column pair]: columns 4 tx + {0,1}, {2,3}, 64 + 4 tx + {0,1}, {2,3}
  uint32_t it = 0;  // k-blocks consumed so far

  for (int tile = cta; tile < ntiles && ok; tile += nctas) {
    int tm, tn;
    tile_to_mn(p, tile, tm, tn);
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.0f, 0.0f);

    for (int kb = 0; kb < p.kblocks; ++kb, ++it) {
      // keep the load stream ahead: refill the stage that was released one k-block ago
      if (!issue_next()) { ok = false; break; }
      const uint32_t s = it % STAGES;
      const uint32_t ph = (it / STAGES) & 1u;
      if (!wait_bounded(full_bar + 8 * s, ph, abort_flag, p)) { ok = false; break; }
      const uint32_t st = tiles_u32 + s * STAGE_BYTES;
      // Four k values per loop iteration, as two pairs (the fully unrolled stage, 2200 instructions,
      // overflowed the instruction cache; 16-byte A fragments for four k at once cost 16 more
      // registers than the 128 that two CTAs per SM allow, and spilled).
#pragma unroll 2
      for (int kp = 0; kp < TK / 2; ++kp) {
        float2 a[RPT];
        const uint32_t ao = st + a_off + ((((uint32_t)kp >> 1) ^ a_sw) << 4) + (((uint32_t)kp & 1u) << 3);
#pragma unroll
        for (int i = 0; i < RPT; ++i) a[i] = lds64_f32(ao + i * 2048);
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
          const uint32_t k7 = (2u * (uint32_t)kp + kk) & 7u;
          const uint32_t bo = st + b_off + (2 * kp + kk) * 128 + ((b_ch ^ k7) << 4);
          const float4 b0 = lds128_f32(bo);
          const float4 b1 = lds128_f32(bo + 2 * B_BOX_BYTES);
#pragma unroll
          for (int i = 0; i < RPT; ++i) {
            // packed FP32 FMA (two independent IEEE fused multiply-adds per instruction): half the
            // issue slots of scalar FFMA for the same arithmetic
            const float2 aa = dup_f32x2(kk == 0 ? a[i].x : a[i].y);
            acc[i][0] = __ffma2_rn(aa, make_float2(b0.x, b0.y), acc[i][0]);
            acc[i][1] = __ffma2_rn(aa, make_float2(b0.z, b0.w), acc[i][1]);
            acc[i][2] = __ffma2_rn(aa, make_float2(b1.x, b1.y), acc[i][2]);
            acc[i][3] = __ffma2_rn(aa, make_float2(b1.z, b1.w), acc[i][3]);
          }
        }
      }
      // Release the stage. The refill writes through the asynchronous proxy, the loads above read
      // through the generic proxy: fence, synchronise the warp, one arrival per warp.
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + 8 * s);
    }
    if (!ok) break;

    // Epilogue: C += acc, 16-byte accesses where the row segment is aligned and inside N.
    const bool vec = ((reinterpret_cast<uintptr_t>(p.C) & 15) == 0) && ((p.ldc & 3) == 0);
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
      const int row = tm * TM + ty + 16 * i;
      if (row >= p.M) continue;
      float* crow = p.C + (long long)row * p.ldc;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int col = tn * TN + 64 * h + 4 * tx;
        if (vec && col + 3 < p.N) {
          float4 c = *reinterpret_cast<const float4*>(crow + col);
          c.x += acc[i][2 * h + 0].x;
          c.y += acc[i][2 * h + 0].y;
          c.z += acc[i][2 * h + 1].x;
          c.w += acc[i][2 * h + 1].y;
          *reinterpret_cast<float4*>(crow + col) = c;
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (col + e < p.N) crow[col + e] += (e & 1) ? acc[i][2 * h + (e >> 1)].y : acc[i][2 * h + (e >> 1)].x;
        }
      }
    }
  }

  // Leaving. After a normal run every copy that was issued has been consumed. After an abort,
  // copies may still be in flight into this CTA's shared memory: let them land first (bounded).
  if (!ok && tid == 0) {
    const uint32_t n_inflight = lit < (uint32_t)STAGES ? lit : (uint32_t)STAGES;
    for (uint32_t q = lit - n_inflight; q < lit; ++q) {
      const uint32_t s = q % STAGES, ph = (q / STAGES) & 1u;
      const unsigned long long t0 = globaltimer_ns();
      while (!mbar_try_wait(full_bar + 8 * s, ph)) {
        if (globaltimer_ns() - t0 > p.wait_limit_ns) break;
      }
    }
  }
  __syncthreads();
}

// Copies a rows x cols float matrix into a 16-byte aligned buffer whose leading dimension is a
// multiple of 32 floats (operands TMA cannot address: base not 16-byte aligned or a leading
// dimension that is not a multiple of 4). One thread per element of a row chunk; gridDim.y may be capped.
__global__ void sgemm_pack_kernel(const float* __restrict__ src, long long ld_src, int rows, int cols,
                                  float* __restrict__ dst, long long ld_dst) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= cols) return;
  for (int r = blockIdx.y; r < rows; r += gridDim.y) dst[(long long)r * ld_dst + c] = src[(long long)r * ld_src + c];
}

}  // namespace sgemm
