// Single-precision C += A*B for sm_100a: exact binary32 arithmetic on the FP32 pipe, fed by the
// same TMA + mbarrier staging as the FP64 kernels. The paper's SGEMM (Section 2.13) is its DGEMM
// nest with f64 replaced by f32 and a wider register tile; here the register tile is 16 x 8 per
// thread (8 x 8 in the 128-row form), the CTA tile 256 x 128 x 32 (128 x 128 x 32), 256 threads,
// one CTA per SM, persistent over the tiles with a stream-K tail.
//
// The FP32 pipe issues one warp-wide instruction per scheduler per clock (128 FMA/clk/SM with
// scalar FMAs), so the bound is instruction issue. The packed fma.rn.f32x2 performs two independent
// IEEE FMAs per instruction and halves the issue slots per flop: per 2 k values a thread issues
// 128 packed FMAs (64 in the 128-row form), 16 (8) 8-byte A loads and 4 16-byte B loads.
#pragma once

#include <cstdint>
#include <cuda.h>

#include "ptx.cuh"

namespace sgemm {

using namespace dgemm::ptx;

// Tile heights: 256 rows (16 x 8 outputs per thread), and 128 or 64 rows (8 x 8, 4 x 8 per thread)
// for problems whose M would leave much of a taller tile empty. Tile widths: 128 columns, or 64
// (NH = 1: each thread keeps only the first of its two groups of four columns) for a narrow N.
// One CTA per SM in every form.
constexpr int TN = 128;  // CTA tile columns of the wide form; row pitch of a workspace slot
constexpr int TK = 32;   // k extent of a stage: 32 floats = one 128-byte swizzle row
constexpr int THREADS = 256;
constexpr int WARPS = THREADS / 32;
constexpr int B_BOX_BYTES = TK * 32 * 4;    // 4 KiB: [32 k][32 columns]
constexpr int LOOKAHEAD = 2;                // k-blocks in flight ahead of the arithmetic
constexpr int SMEM_ALIGN = 1024;
constexpr int MAX_TM = 256;                 // a workspace slot holds MAX_TM x TN floats

template <int RPT, int NH = 2>
struct Cfg {
  static constexpr int TM = 16 * RPT;                 // CTA tile rows
  static constexpr int TNV = 64 * NH;                 // CTA tile columns
  static constexpr int A_BYTES = TM * TK * 4;         // rows of 128 bytes
  static constexpr int B_BYTES = (TNV / 32) * B_BOX_BYTES;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = 4;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SMEM_ALIGN + 256;
};
constexpr int STATUS_TIMEOUT = -8;          // DGEMM_ERR_TIMEOUT


struct Params {
  int M, N, K;
  int tiles_m, tiles_n;
  int kblocks;         // ceil(K / TK)
  int group_m;         // raster group height in tiles
  int b_blocked_map;   // map_b is the 3-D view (32 columns, K, N/32): one copy stages the whole B tile
  // Work decomposition (as in the FP64 kernels): tiles [0, dp_tiles) run whole, CTA b taking b,
  // b + G, ...; the k-blocks of the remaining tail_tiles are cut into equal spans of tail_ipc, one
  // per CTA. A span covers at most two tile segments; a segment that is not a whole tile goes to
  // workspace slot 2 * cta + j and sgemm_tail_reduce_kernel adds the slots to C in CTA order.
  int dp_tiles, tail_tiles, tail_ipc;
  float* partial;      // workspace: slots of MAX_TM * TN floats
  int tm_rows;         // rows of a CTA tile (256, 128 or 64)
  int tn_cols;         // columns of a CTA tile (128 or 64)
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

struct Item {
  int tile, kb0, kb1;  // tile and k-block range [kb0, kb1)
  int slot;            // workspace slot for the partial tile, or -1: add straight into C
};

// The idx-th work item of CTA `cta`; false past the end of its list.
__device__ __forceinline__ bool get_item(const Params& p, int cta, int nctas, int idx, Item& w) {
  const int n1 = cta < p.dp_tiles ? (p.dp_tiles - cta + nctas - 1) / nctas : 0;
  if (idx < n1) {
    w.tile = cta + idx * nctas;
    w.kb0 = 0;
    w.kb1 = p.kblocks;
    w.slot = -1;
    return true;
  }
  const int j = idx - n1;
  if (j > 1 || p.tail_tiles == 0) return false;
  const int total = p.tail_tiles * p.kblocks;  // the host keeps this below 2^31
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
  w.tile = p.dp_tiles + trel;
  w.kb0 = s0 - trel * p.kblocks;
  w.kb1 = s1 - trel * p.kblocks;
  w.slot = (w.kb0 == 0 && w.kb1 == p.kblocks) ? -1 : 2 * cta + j;
  return true;
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

template <int RPT, int NH>
__global__ void __launch_bounds__(THREADS, 1)
sgemm_ffma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ Params p) {
  constexpr int TM = Cfg<RPT, NH>::TM;
  constexpr int TNV = Cfg<RPT, NH>::TNV;
  constexpr int A_BYTES = Cfg<RPT, NH>::A_BYTES;
  constexpr int STAGE_BYTES = Cfg<RPT, NH>::STAGE_BYTES;
  constexpr int STAGES = Cfg<RPT, NH>::STAGES;
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
  grid_dependency_wait();  // launched with programmatic serialization: the set-up above overlaps the previous kernel's tail

  const int cta = blockIdx.x, nctas = gridDim.x;

  // Load stream: the k-blocks of this CTA's work items in order, LOOKAHEAD k-blocks ahead of the
  // arithmetic and across item boundaries. Every thread follows the cursor; k-block number i is
  // issued by lane 0 of warp i mod 8.
  int l_idx = 0, l_kb = 0, l_kb1 = 0, l_tm = 0, l_tn = 0;
  bool l_valid;
  auto cursor_load = [&]() {
    Item li;
    l_valid = get_item(p, cta, nctas, l_idx, li);
    if (l_valid) {
      l_kb = li.kb0;
      l_kb1 = li.kb1;
      tile_to_mn(p, li.tile, l_tm, l_tn);
    }
  };
  cursor_load();
  uint32_t lit = 0;
  auto issue_next = [&]() -> bool {
    if (!l_valid) return true;
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
            tma_load_3d(sb, &map_b, 0, l_kb * TK, l_tn * (TNV / 32), fb);
          } else {
            for (int nb = 0; nb < TNV / 32; ++nb) tma_load_2d(sb + nb * B_BOX_BYTES, &map_b, l_tn * TNV + nb * 32, l_kb * TK, fb);
          }
        } else {
          good = 0;
        }
      }
      if (!__all_sync(0xffffffffu, good)) return false;
    }
    ++lit;
    if (++l_kb >= l_kb1) {
      ++l_idx;
      cursor_load();
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

  float2 acc[RPT][2 * NH];  // [row i][column pair]: columns 4 tx + {0,1}, {2,3} and, in the wide form, 64 + 4 tx + {0,1}, {2,3}
  uint32_t it = 0;  // k-blocks consumed so far

  for (int idx = 0; ok; ++idx) {
    Item w;
    if (!get_item(p, cta, nctas, idx, w)) break;
    int tm, tn;
    tile_to_mn(p, w.tile, tm, tn);
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
      for (int j = 0; j < 2 * NH; ++j) acc[i][j] = make_float2(0.0f, 0.0f);

    for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
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
          float4 b1 = b0;
          if constexpr (NH == 2) b1 = lds128_f32(bo + 2 * B_BOX_BYTES);
#pragma unroll
          for (int i = 0; i < RPT; ++i) {
            // packed FP32 FMA (two independent IEEE fused multiply-adds per instruction): half the
            // issue slots of scalar FFMA for the same arithmetic
            const float2 aa = dup_f32x2(kk == 0 ? a[i].x : a[i].y);
            acc[i][0] = __ffma2_rn(aa, make_float2(b0.x, b0.y), acc[i][0]);
            acc[i][1] = __ffma2_rn(aa, make_float2(b0.z, b0.w), acc[i][1]);
            if constexpr (NH == 2) {
              acc[i][2] = __ffma2_rn(aa, make_float2(b1.x, b1.y), acc[i][2]);
              acc[i][3] = __ffma2_rn(aa, make_float2(b1.z, b1.w), acc[i][3]);
            }
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

    if (w.slot >= 0) {
      // a segment of a tail tile: the partial sums go to the workspace (row-major TM x TN)
      float* dst = p.partial + (long long)w.slot * (MAX_TM * TN);
#pragma unroll
      for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int h = 0; h < NH; ++h)
          *reinterpret_cast<float4*>(dst + (ty + 16 * i) * TN + 64 * h + 4 * tx) =
              make_float4(acc[i][2 * h].x, acc[i][2 * h].y, acc[i][2 * h + 1].x, acc[i][2 * h + 1].y);
      continue;
    }
    // Epilogue: C += acc, 16-byte accesses where the row segment is aligned and inside N, else 4-byte
    // accesses with a bounds check per element. Four rows at a time, all their loads issued before
    // the first store (interleaved, every load would wait for the store before it, which may alias
    // as far as the compiler knows, and an edge tile would cost one memory latency per element).
    const bool vec = ((reinterpret_cast<uintptr_t>(p.C) & 15) == 0) && ((p.ldc & 3) == 0);
#pragma unroll
    for (int i0 = 0; i0 < RPT; i0 += 4) {
      float4 cin[4][NH];
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) {
        const int row = tm * TM + ty + 16 * (i0 + ii);
        const float* crow = p.C + (long long)row * p.ldc;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          const int col = tn * TNV + 64 * h + 4 * tx;
          if (row < p.M && vec && col + 3 < p.N) {
            cin[ii][h] = *reinterpret_cast<const float4*>(crow + col);
          } else {
            cin[ii][h].x = (row < p.M && col + 0 < p.N) ? crow[col + 0] : 0.0f;
            cin[ii][h].y = (row < p.M && col + 1 < p.N) ? crow[col + 1] : 0.0f;
            cin[ii][h].z = (row < p.M && col + 2 < p.N) ? crow[col + 2] : 0.0f;
            cin[ii][h].w = (row < p.M && col + 3 < p.N) ? crow[col + 3] : 0.0f;
          }
        }
      }
#pragma unroll
      for (int ii = 0; ii < 4; ++ii) {
        const int i = i0 + ii;
        const int row = tm * TM + ty + 16 * i;
        if (row >= p.M) continue;
        float* crow = p.C + (long long)row * p.ldc;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          const int col = tn * TNV + 64 * h + 4 * tx;
          float4 c = cin[ii][h];
          c.x += acc[i][2 * h + 0].x;
          c.y += acc[i][2 * h + 0].y;
          c.z += acc[i][2 * h + 1].x;
          c.w += acc[i][2 * h + 1].y;
          if (vec && col + 3 < p.N) {
            *reinterpret_cast<float4*>(crow + col) = c;
          } else {
            if (col + 0 < p.N) crow[col + 0] = c.x;
            if (col + 1 < p.N) crow[col + 1] = c.y;
            if (col + 2 < p.N) crow[col + 2] = c.z;
            if (col + 3 < p.N) crow[col + 3] = c.w;
          }
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

// Adds the partial tiles of tail tile blockIdx.x to C: C[i][j] += ((p_0 + p_1) + ...) in the order of
// the CTAs that computed them. Deterministic. blockIdx.y takes TM / 16 consecutive rows.
__global__ void sgemm_tail_reduce_kernel(const Params p) {
  grid_dependency_wait();
  const int trel = blockIdx.x;
  const int lo = trel * p.kblocks, hi = lo + p.kblocks;
  const int c_first = lo / p.tail_ipc, c_last = (hi - 1) / p.tail_ipc;
  if (c_first == c_last) return;  // one CTA had the whole tile and added it straight to C
  int tm, tn;
  tile_to_mn(p, p.dp_tiles + trel, tm, tn);
  const int TM = p.tm_rows;
  const int chunk = TM * TN / 16;
  const int e0 = blockIdx.y * chunk;
  for (int e = e0 + 4 * threadIdx.x; e < e0 + chunk; e += 4 * blockDim.x) {
    const int r = e / TN, c = e - r * TN;  // (a slot's rows are TN floats apart in either form)
    const int row = tm * TM + r, col = tn * p.tn_cols + c;
    if (row >= p.M || c >= p.tn_cols || col >= p.N) continue;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int cta = c_first; cta <= c_last; ++cta) {
      const int slot = 2 * cta + ((cta * p.tail_ipc >= lo) ? 0 : 1);
      const float4 v = *reinterpret_cast<const float4*>(p.partial + (long long)slot * (MAX_TM * TN) + e);
      if (cta == c_first) {
        sum = v;
      } else {
        sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
      }
    }
    float* dst = p.C + (long long)row * p.ldc + col;
    dst[0] += sum.x;
    if (col + 1 < p.N) dst[1] += sum.y;
    if (col + 2 < p.N) dst[2] += sum.z;
    if (col + 3 < p.N) dst[3] += sum.w;
  }
}

// Copies a rows x cols float matrix into a 16-byte aligned buffer whose leading dimension is a
// multiple of 32 floats (operands TMA cannot address: base not 16-byte aligned or a leading
// dimension that is not a multiple of 4). One thread per element of a row chunk; gridDim.y may be capped.
// One or two operands per launch (blockIdx.z selects; blocks beyond the smaller operand's extent
// return at once). Launched with programmatic stream serialization: waits for the kernel before
// it, which may still be reading the scratch this one writes.
struct PackOpF {
  const float* src;
  long long ld_src;
  int rows, cols;
  float* dst;
  long long ld_dst;
};
__global__ void sgemm_pack_kernel(const PackOpF a, const PackOpF b) {
  grid_dependency_wait();
  const PackOpF& o = blockIdx.z == 0 ? a : b;
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= o.cols) return;
  for (int r = blockIdx.y; r < o.rows; r += gridDim.y) o.dst[(long long)r * o.ld_dst + c] = o.src[(long long)r * o.ld_src + c];
}

}  // namespace sgemm
