// Split-K inside a thread-block cluster, for problems too small to fill the GPU with whole tiles.
//
// A problem of a few tiles only reaches all SMs when K is cut as well. The general kernels do that
// through a workspace in global memory and a second (reduction) kernel; on a problem of a few
// microseconds that second launch and the round trip through L2 are a large share of the time.
// Here the S CTAs that share one 64 x 128 tile of C form a cluster (S = 1, 2, 4 or 8): CTA r
// multiplies k-blocks [r * kps, (r + 1) * kps), leaves its partial tile in its own shared memory
// (in the space of the operand stages, which are dead by then), the cluster synchronises, and
// CTA r then adds rows [r * 64 / S, (r + 1) * 64 / S) of all S partial tiles in rank order, read
// through distributed shared memory, into C. One launch, no workspace, and the result is that of
// the workspace path with the same K partition, bit for bit:
//     C = beta * C + alpha * (((p_0 + p_1) + p_2) + ...).
//
// The cluster barrier is a hardware barrier without a time limit, so every thread of every CTA
// reaches both of its instances on every path, also after a bounded wait has given up (the CTA
// then skips the arithmetic and the status word reports the timeout).
#pragma once

#include "dgemm_dmma.cuh"

namespace dgemm {

constexpr int CLUSTER_MAX = 8;  // portable cluster size limit

// One stage (A: TBM x 16, B: 16 x TBN doubles, the swizzled layout of the TMA copies) staged with
// 8-byte asynchronous copies, zero fill outside the matrices: any alignment, any leading dimension.
// A: 16 consecutive threads copy the 16 k values of one row; B: TBN consecutive threads copy TBN
// consecutive columns of one k row.
template <int TBM, int TBN, int THREADS>
__device__ __forceinline__ void stage_copy_generic(const GemmParams& p, uint32_t sa, uint32_t sb, int m0, int n0, int k0, int tid) {
  {
    const int a_k = tid & 15, row0 = tid >> 4;
    const int k = k0 + a_k;
    const bool kin = k < p.K;
    const double* src = p.A + (long long)(m0 + row0) * p.lda + k;
    const uint32_t dst_base = sa + ((a_k & 1) << 3);
    constexpr int ROW_STEP = THREADS / 16;
#pragma unroll
    for (int i = 0; i < TBM / ROW_STEP; ++i) {
      const int row = row0 + ROW_STEP * i;
      const bool in = kin && (m0 + row < p.M);
      const uint32_t dst = dst_base + row * 128 + (((a_k >> 1) ^ (row & 7)) << 4);
      ptx::cp_async_8(dst, in ? (const void*)(src + (long long)(ROW_STEP * i) * p.lda) : (const void*)p.A, in ? 8u : 0u);
    }
  }
  {
    const int nn = tid % TBN, kk0 = tid / TBN;
    const bool nin = n0 + nn < p.N;
    const double* src = p.B + (long long)(k0 + kk0) * p.ldb + (n0 + nn);
    const uint32_t dst_base = sb + (nn >> 4) * B_BOX_BYTES + ((nn & 1) << 3);
    const int chunk = (nn & 15) >> 1;
    constexpr int K_STEP = THREADS / TBN;
#pragma unroll
    for (int i = 0; i < BK / K_STEP; ++i) {
      const int kk = kk0 + K_STEP * i;
      const bool in = nin && (k0 + kk < p.K);
      const uint32_t dst = dst_base + kk * 128 + ((chunk ^ (kk & 7)) << 4);
      ptx::cp_async_8(dst, in ? (const void*)(src + (long long)(K_STEP * i) * p.ldb) : (const void*)p.B, in ? 8u : 0u);
    }
  }
}

// BT / AT (TMA staging only): B / A is the matrix as stored, N x K / K x M, and the transposed tile is
// staged by the copy engine itself, as in the inline kernel's 64 x 128 tile.
template <bool USE_TMA, int TBM, int WTM = 64, int TBN = BN, bool BT = false, bool AT = false>
__global__ void __launch_bounds__(TileCfg<TBM, WTM, TBN>::THREADS_, 2)
dgemm_cluster_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                     const __grid_constant__ GemmParams p) {
  using Cfg = TileCfg<TBM, WTM, TBN>;
  constexpr int MT = Cfg::MT_;
  constexpr int WARPS_N = Cfg::WARPS_N;
  constexpr int STAGES = Cfg::STAGES_;
  constexpr int LOOKAHEAD = Cfg::LOOKAHEAD_;
  constexpr int WARPS = Cfg::WARPS_;
  constexpr int THREADS = Cfg::THREADS_;
  constexpr int A_STAGE_BYTES = Cfg::A_BYTES;
  constexpr int STAGE_BYTES = Cfg::STAGE_BYTES_;
  constexpr int RED_STRIDE = TBN * 8 + 16;  // bytes per row of the partial tile in shared memory (16 of padding)
  constexpr int PAIRS_ROW = TBN / 2;
  constexpr int U = 4;                      // element pairs per thread and pass of the reduction (8 was slower)
  static_assert(Cfg::CTAS_PER_SM == 2, "the cluster kernel is built for the two-CTAs-per-SM tiles");
  static_assert(TBM * RED_STRIDE <= STAGES * STAGE_BYTES, "the partial tile must fit in the stage area");
  static_assert(TBM % CLUSTER_MAX == 0, "every rank reduces a whole number of rows");
  static_assert(USE_TMA || (!BT && !AT), "transposed operands are staged in place by the copy engine only");

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + STAGES * STAGE_BYTES);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES);
  const uint32_t tiles_u32 = raw + pad;  // the same offset in every CTA of the cluster (same kernel, same launch)
  const uint32_t full_bar = tiles_u32 + STAGES * STAGE_BYTES;
  const uint32_t empty_bar = full_bar + 8 * STAGES;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int S = (int)ptx::cluster_nctarank();
  const int rank = (int)ptx::cluster_ctarank();

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar + 8 * s, USE_TMA ? 1 : THREADS);
      ptx::mbar_init(empty_bar + 8 * s, WARPS);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    if (USE_TMA) {
      ptx::prefetch_tensormap(&map_a);
      ptx::prefetch_tensormap(&map_b);
    }
  }
  __syncthreads();
  ptx::grid_dependency_wait();

  int tm, tn;
  tile_to_mn(p, (int)blockIdx.x / S, tm, tn);
  const int kb0 = min(rank * p.kblocks_per_split, p.kblocks);
  const int nkb = min(kb0 + p.kblocks_per_split, p.kblocks) - kb0;  // k-blocks of this CTA (0 for a rank beyond the last partition)
  const int n_act = (p.kblocks + p.kblocks_per_split - 1) / p.kblocks_per_split;  // ranks that hold a partial tile
  const int rows_per = TBM / S;
  const int row_first = rank * rows_per;  // rows of the tile this CTA reduces

  // The copies of k-block j of this CTA into stage j % STAGES. TMA staging: issued by lane 0 of
  // warp 0; generic staging: every thread copies its share.
  auto issue = [&](int j) -> bool {
    const uint32_t s = (uint32_t)j % STAGES, ph = ((uint32_t)j / STAGES) & 1u;
    if (!wait_bounded<false>(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) return false;
    const uint32_t sa = tiles_u32 + s * STAGE_BYTES, sb = sa + A_STAGE_BYTES, fb = full_bar + 8 * s;
    if (p.drop_loads) return true;  // testing aid: nothing is copied, the waits on this stage run out
    if (!USE_TMA) {
      stage_copy_generic<TBM, TBN, THREADS>(p, sa, sb, tm * TBM, tn * TBN, (kb0 + j) * BK, tid);
      ptx::cp_async_mbar_arrive_noinc(fb);
      return true;
    }
    ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
    if constexpr (AT) {
      tma_load_at(sa, &map_a, p.a_blocked_map, tm * TBM, (kb0 + j) * BK, fb, TBM / 16);
    } else {
      ptx::tma_load_2d(sa, &map_a, (kb0 + j) * BK, tm * TBM, fb);
    }
    if constexpr (BT) {
      ptx::tma_load_2d(sb, &map_b, (kb0 + j) * BK, tn * TBN, fb);  // rows n of B^T, 16 k each
    } else if (p.b_blocked_map) {
      ptx::tma_load_3d(sb, &map_b, 0, (kb0 + j) * BK, tn * (TBN / 16), fb);
    } else {
      tma_load_b_boxes(sb, &map_b, tn * TBN, (kb0 + j) * BK, fb, TBN / 16);
    }
    return true;
  };

  bool ok = true;
  int issued = 0;  // TMA staging: meaningful in lane 0 of warp 0 only
  if (!USE_TMA) {
    for (; issued < nkb && issued < LOOKAHEAD && ok; ++issued) ok = __all_sync(0xffffffffu, issue(issued) ? 1 : 0);
  } else if (warp == 0) {
    int good = 1;
    if (lane == 0) {
      for (; issued < nkb && issued < LOOKAHEAD && good; ++issued) good = issue(issued) ? 1 : 0;
    }
    ok = __all_sync(0xffffffffu, good);
  }

  // The elements of C this thread will update, as pairs (row, col), (row, col + 1): pair number
  // q of the CTA's rows_per x TBN slice is handled by thread q % THREADS in pass q / (THREADS * U).
  // The old values of the first pass are loaded now, long before they are needed (with S = 8 that
  // is the only pass); the rows of the later passes are requested into L2.
  const int total_pairs = rows_per * PAIRS_ROW;
  double cx[U], cy[U];
  long long off[U];
  uint32_t src[U];
  bool in0[U], in1[U];
  auto locate = [&](int q0) {
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int q = q0 + THREADS * u;
      const int r = row_first + q / PAIRS_ROW, c = 2 * (q % PAIRS_ROW);
      const int row = tm * TBM + r, col = tn * TBN + c;
      in0[u] = q < total_pairs && row < p.M && col < p.N;
      in1[u] = in0[u] && col + 1 < p.N;
      off[u] = (long long)row * p.ldc + col;
      src[u] = tiles_u32 + r * RED_STRIDE + c * 8;
      cx[u] = (p.load_c && in0[u]) ? p.C[off[u]] : -0.0;
      cy[u] = (p.load_c && in1[u]) ? p.C[off[u] + 1] : -0.0;
    }
  };
  locate(tid);
  if (p.load_c && total_pairs > THREADS * U) {
    for (int i = tid; i < rows_per * (TBN / 16); i += THREADS) {
      const int row = tm * TBM + row_first + i / (TBN / 16), col = tn * TBN + 16 * (i % (TBN / 16));
      if (row < p.M && col < p.N) ptx::prefetch_l2(p.C + (long long)row * p.ldc + col);
    }
  }

  const LaneMap lm = make_lane_map(warp, lane, A_STAGE_BYTES, WTM, WARPS_N, BT, AT);
  double acc[MT][4][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int c = 0; c < 4; ++c) acc[mt][nt][c] = 0.0;

  for (int i = 0; i < nkb && ok; ++i) {
    const uint32_t s = (uint32_t)i % STAGES, ph = ((uint32_t)i / STAGES) & 1u;
    // Every decision to leave the loop is taken by the whole warp (a vote per wait: this kernel only
    // runs problems of a few k-blocks), so no lane can be left behind in a warp-level
    // synchronisation and every warp reaches the CTA and cluster barriers below.
    const bool arrived = wait_bounded(full_bar + 8 * s, ph, abort_flag, p);
    if (!__all_sync(0xffffffffu, arrived ? 1 : 0)) { ok = false; break; }
    compute_kblock<false, MT, BT, AT>(tiles + s * STAGE_BYTES, lm, acc);
    release_stage(empty_bar + 8 * s, lane);
    if (!USE_TMA) {
      if (i + LOOKAHEAD < nkb && !__all_sync(0xffffffffu, issue(i + LOOKAHEAD) ? 1 : 0)) { ok = false; break; }
    } else if (warp == 0 && i + LOOKAHEAD < nkb) {  // refill the stage all warps released two k-blocks ago
      int good = 1;
      if (lane == 0) {
        good = issue(i + LOOKAHEAD) ? 1 : 0;
        issued += good;
      }
      if (!__all_sync(0xffffffffu, good)) { ok = false; break; }
    }
  }

  if (!USE_TMA) ptx::cp_async_wait_all();
  __syncthreads();  // every warp is done with the stages
  ok = (*abort_flag == 0);  // uniform over the CTA from here on

  // This CTA's partial tile, row-major, over the stage area.
  if (ok && nkb > 0) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int half = 0; half < 2; ++half)
#pragma unroll
        for (int np = 0; np < 2; ++np) {
          const int r = lm.row0 + lm.rm + 16 * mt + 8 * half;
          const int c = 32 * lm.wn + 4 * lm.t + 16 * np;
          const uint32_t dst = tiles_u32 + r * RED_STRIDE + c * 8;
          ptx::sts128(dst, acc[mt][2 * np][2 * half], acc[mt][2 * np + 1][2 * half]);
          ptx::sts128(dst + 16, acc[mt][2 * np][2 * half + 1], acc[mt][2 * np + 1][2 * half + 1]);
        }
  }
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();

  if (ok) {
    for (int q0 = tid; q0 < total_pairs; q0 += THREADS * U) {
      double sx[U], sy[U];
      if (q0 != tid) locate(q0);
      // Partial tiles are read four ranks at a time, all of a batch's loads issued before the first
      // addition (a remote shared-memory read is a round trip through the cluster's network). The
      // additions keep rank order. (512^3: 18.7 -> 18.2 us.)
#pragma unroll
      for (int s0 = 0; s0 < CLUSTER_MAX; s0 += 4) {
        if (s0 < n_act) {
          double vx[4][U], vy[4][U];
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (s0 + j < n_act) {
#pragma unroll
              for (int u = 0; u < U; ++u) ptx::ld_cluster_128(ptx::map_to_cta(src[u], (uint32_t)(s0 + j)), vx[j][u], vy[j][u]);
            }
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (s0 + j < n_act) {
#pragma unroll
              for (int u = 0; u < U; ++u) {
                if (s0 + j == 0) {
                  sx[u] = vx[j][u];
                  sy[u] = vy[j][u];
                } else {
                  sx[u] += vx[j][u];
                  sy[u] += vy[j][u];
                }
              }
            }
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const double ax = sx[u] * p.alpha, ay = sy[u] * p.alpha;  // exact for alpha == 1
        if (in0[u]) p.C[off[u]] = p.load_c ? fma(cx[u], p.beta, ax) : ax;
        if (in1[u]) p.C[off[u] + 1] = p.load_c ? fma(cy[u], p.beta, ay) : ay;
      }
    }
  }
  // no CTA leaves (and gives up its shared memory) while another may still be reading it
  ptx::cluster_arrive_release();
  ptx::cluster_wait_acquire();

  // After an abort, copies may still be in flight into this CTA's shared memory: let them land.
  if (USE_TMA && !ok && !p.drop_loads && tid == 0) {
    const int first = issued > STAGES ? issued - STAGES : 0;
    for (int q = first; q < issued; ++q) {
      const uint32_t s = (uint32_t)q % STAGES, ph = ((uint32_t)q / STAGES) & 1u;
      const unsigned long long t0 = ptx::globaltimer_ns();
      while (!ptx::mbar_try_wait(full_bar + 8 * s, ph)) {
        if (ptx::globaltimer_ns() - t0 > DRAIN_LIMIT_NS) break;
      }
    }
  }
  __syncthreads();
}

}  // namespace dgemm
