// Warp-specialised FP64 GEMM kernel whose epilogue leaves the SM asynchronously: for problems with
// a short K (rank-k updates, the BLIS macro-kernel shape), where a tile's few k-blocks cannot hide a
// round trip of its C tile through the registers of the warps that also do the arithmetic.
//
// Same producer warpgroup, stages, fragment layout and software-pipelined consumer loop as
// dgemm_dmma_ws_kernel<true, 128> (128 x 128 tiles, one CTA per SM), with three differences:
//   * five stages instead of six; the shared memory saved holds half a C tile (64 rows x 128
//     columns, 64 KB): the tile buffer;
//   * the consumer warps do not load C. The four warps of a 64-row slab write their accumulators
//     into the tile buffer (row-major, 1024 bytes per row; lanes with even and odd row group store
//     their two 16-byte pieces in opposite order, which keeps the stores free of bank conflicts),
//     and an otherwise idle warp of the producer warpgroup hands the buffer to the copy engine, two
//     rows per lane: a bulk REDUCE (add.f64) of 1024 contiguous bytes into the row of C for
//     beta == 1, a bulk STORE for beta == 0. The addition C + acc happens at the L2 (one rounding,
//     exactly the c + acc of the other epilogues), and the arithmetic of the next tile starts as
//     soon as the buffer is written. Whole-row requests measured faster than tiled boxes of 16
//     columns through a tensor map (a pass that only reduces 16384^2 doubles: 806 against 919 us),
//     and asking L2 for the C tile ahead of the reduce, as the other kernels' epilogues do, made
//     this one slower (K = 64: 1084 -> 1040 us): both together 16384^2 x 64 1084 -> 1024 us,
//     x 16 1075 -> 865 us. A request cannot clip a row, so the tiles of a ragged last tile column
//     are added to C by the consumer warps themselves, like in the other kernels. (Issued by a
//     consumer warp, the copy instructions and the waits around them put that warp 1 - 2 k cycles
//     behind its neighbours on every tile, and they then waited for it.)
//   * the two slabs of a tile take turns with the one buffer: slab 0 of tile t, slab 1 of tile t,
//     slab 0 of tile t + 1, ... A slab writes once the copy engine has read the previous user's data
//     (cp.async.bulk.wait_group.read in the issuing thread). The turns keep the slabs a few thousand
//     cycles apart for good, and that is wanted: the two warps that share a scheduler belong to
//     different slabs, so one of them multiplies while the other is in its epilogue. The hand-overs
//     (buffer written: four warps -> issuing thread; your turn: issuing thread -> the next four
//     warps, one barrier per slab) are mbarriers with the same bounded waits as the stages, so a
//     warp that gives up cannot leave anybody at a barrier.
// Needs a C the copy engine can address: 16-byte aligned base, even ldc; beta == 0 or 1.
// Partial tiles (stream-K tail, forced split K) go to the workspace as in the other kernels.
#pragma once

#include "dgemm_dmma.cuh"

namespace dgemm {

struct WsBulkCfg {
  static constexpr int STAGES_ = 5;
  static constexpr int CONSUMER_WARPS = 8;
  static constexpr int THREADS_ = (CONSUMER_WARPS + WS_PRODUCER_WARPS) * 32;
  static constexpr int C_ROW_BYTES = BN * 8;                      // a row of the tile buffer
  static constexpr int C_BUF_BYTES = 64 * C_ROW_BYTES;            // one slab of a tile: 64 rows x 128 columns, row-major
  static constexpr int C_OFFSET = STAGES_ * STAGE_BYTES;          // from the first stage; a multiple of 1024
  static constexpr int BAR_OFFSET = C_OFFSET + C_BUF_BYTES;
  static constexpr int SMEM_BYTES_ = BAR_OFFSET + SMEM_ALIGN + 1024;  // + alignment slack + barriers, flags, work words
};
static_assert(WsBulkCfg::SMEM_BYTES_ <= 227 * 1024, "stages + C tile must fit the shared memory of one SM");

__global__ void __launch_bounds__(WsBulkCfg::THREADS_, 1)
dgemm_dmma_wsb_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                      const __grid_constant__ GemmParams p) {
  constexpr int STAGES = WsBulkCfg::STAGES_;
  constexpr int WARPS = WsBulkCfg::CONSUMER_WARPS;
  constexpr int TBM = BM;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t pad = (SMEM_ALIGN - (raw & (SMEM_ALIGN - 1))) & (SMEM_ALIGN - 1);
  uint8_t* tiles = smem_raw + pad;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + WsBulkCfg::BAR_OFFSET);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * STAGES + 3);
  volatile int* work_words = abort_flag + 8;  // 8 words per warp (12 warps)
  const uint32_t tiles_u32 = raw + pad;
  const uint32_t full_bar = tiles_u32 + WsBulkCfg::BAR_OFFSET;
  const uint32_t empty_bar = full_bar + 8 * STAGES;
  // Hand-overs of the tile buffer. c_full: written (a slab's 4 warps -> issuing thread), one phase per
  // use. c_turn[s]: slab s may write now (issuing thread -> slab s's 4 warps), one phase per turn of
  // that slab. A barrier per slab, so that no waiter can ever be two phases away from the barrier it
  // polls: a parity wait cannot tell phase n from phase n - 2.
  const uint32_t c_full = empty_bar + 8 * STAGES;
  const uint32_t c_turn = c_full + 8;  // c_turn + 8 * slab
  const uint32_t c_buf = tiles_u32 + WsBulkCfg::C_OFFSET;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(full_bar + 8 * s, 1);
      ptx::mbar_init(empty_bar + 8 * s, WARPS);
    }
    ptx::mbar_init(c_full, 4);
    ptx::mbar_init(c_turn, 1);
    ptx::mbar_init(c_turn + 8, 1);
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
    ptx::setmaxnreg_dec<WS_PRODUCER_REGS>();
    const int pw = warp - WARPS;
    if (pw == 0 && lane == 0) {
      ptx::prefetch_tensormap(&map_a);
      ptx::prefetch_tensormap(&map_b);
    }
    for (int idx = 0; pw == 0 && ok; ++idx) {
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
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % STAGES;
        const uint32_t ph = (it / STAGES) & 1u;
        const uint32_t sa = tiles_u32 + s * STAGE_BYTES;
        const uint32_t sb = sa + A_STAGE_BYTES;
        const uint32_t fb = full_bar + 8 * s;
        int good = 1;
        if (lane == 0) {
          if (!wait_bounded_inline(empty_bar + 8 * s, ph ^ 1u, abort_flag, p)) {
            good = 0;
          } else if (!p.drop_loads) {
            ptx::mbar_arrive_expect_tx(fb, STAGE_BYTES);
            ptx::tma_load_2d(sa, &map_a, kb * BK, w.tm * TBM, fb);
            if (p.b_blocked_map) {
              ptx::tma_load_3d(sb, &map_b, 0, kb * BK, w.tn * (BN / 16), fb);
            } else {
              tma_load_b_boxes_inline(sb, &map_b, w.tn * BN, kb * BK, fb);
            }
          }
        }
        if (!__all_sync(0xffffffffu, good)) { ok = false; break; }
      }
    }
    if (!ok && !p.drop_loads && pw == 0 && lane == 0) {
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
    // Producer warp 1: the copy-engine hand-over. It walks the same list of work items; for a tile
    // that goes straight to C it takes slab 0 and slab 1 in turn: waits until the slab's four consumer
    // warps have written the tile buffer, issues the 64 row copies (two per lane), waits until the
    // copy engine has read the buffer and passes it on.
    if (pw == 1) {
      uint32_t use = 0;  // uses of the tile buffer so far: 2 x tiles + slab
      bool pending = false;
      for (int idx = 0; ok; ++idx) {
        fetch_work_inline(p, cta, nctas, idx, item_words);
        __syncwarp();
        w.tm = item_words[0];
        w.tn = item_words[1];
        w.slot = item_words[4];
        const int valid = item_words[5];
        __syncwarp();
        if (!valid) break;
        if (w.slot >= 0) continue;  // a partial tile: the consumers store it into the workspace themselves
        if (w.tn * BN + BN > p.N) continue;  // a ragged last tile column: the consumers' own epilogue
        for (int slab = 0; slab < 2 && ok; ++slab, ++use) {
          // every lane polls the barrier (it is complete for all or for none soon after) ...
          const int good = wait_bounded_inline(c_full, use & 1u, abort_flag, p) ? 1 : 0;
          if (!__all_sync(0xffffffffu, good)) { ok = false; break; }
          // ... and sends two rows of the slab: 1024 contiguous bytes each
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const int r = lane + 32 * q;
            const int y = w.tm * TBM + 64 * slab + r;
            if (y < p.M) {
              double* dst = p.C + (long long)y * p.ldc + (long long)w.tn * BN;
              if (p.load_c) ptx::bulk_reduce_add_f64(dst, c_buf + (uint32_t)(r * WsBulkCfg::C_ROW_BYTES), WsBulkCfg::C_ROW_BYTES);
              else ptx::bulk_store(dst, c_buf + (uint32_t)(r * WsBulkCfg::C_ROW_BYTES), WsBulkCfg::C_ROW_BYTES);
            }
          }
          ptx::bulk_commit_group();
          pending = true;
          ptx::bulk_wait_group_read_all();  // the copy engine has read this lane's rows
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(c_turn + 8 * ((use + 1) & 1u));  // the other slab's turn
        }
      }
      if (pending) ptx::bulk_wait_group_all();  // nothing of this CTA is in flight when it leaves
    }
  } else {
    // ------------------------------------------------------------------ consumer warps
    ptx::setmaxnreg_inc<WS_CONSUMER_REGS>();
    const LaneMap lm = make_lane_map(warp, lane, A_STAGE_BYTES, 64, 4);
    // This lane's place in the tile buffer, which holds one slab (64 rows) row-major. The lane owns
    // rows rm + 8 j (j < 8) and, in each, columns 32 wn + 16 np + 4t .. + 3 (np < 2): two 16-byte pieces.
    // Lanes of a quarter-warp with even and odd g write rows that differ by 4, i.e. by a multiple of
    // 128 bytes; storing the two pieces in opposite order in the two kinds of lanes keeps every
    // 16-byte store free of bank conflicts.
    const int slab = lm.wm;
    const bool swap = (lm.g & 1) != 0;
    const uint32_t c_lane = c_buf + (uint32_t)(lm.rm * WsBulkCfg::C_ROW_BYTES) + (uint32_t)(32 * lm.wn + 4 * lm.t) * 8u;
    const uint32_t ch_first = swap ? 16u : 0u;
    const uint32_t ch_second = swap ? 0u : 16u;
    uint32_t use = (uint32_t)slab;         // this slab's next turn with the tile buffer: 2 x tiles so far + slab
    double acc[4][4][4];
    // The work item of the next tile is looked up while the last k-block of the current one is
    // multiplied (its integer divisions then hide behind the MMAs instead of standing between two tiles).
    Work wn;
    bool have = get_work(p, cta, nctas, 0, w);
    for (int idx = 0; ok && have; ++idx, w = wn) {
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
        load_frags<0>(f0, tiles_u32 + s * STAGE_BYTES, lm);
      }
      for (int kb = w.kb0; kb < w.kb1; ++kb, ++it) {
        const uint32_t s = it % STAGES;
        const uint32_t s1 = (it + 1) % STAGES;
        const uint32_t ph1 = ((it + 1) / STAGES) & 1u;
        const bool more = kb + 1 < w.kb1;
        const bool ready = more && ptx::mbar_test_wait(full_bar + 8 * s1, ph1);
        mma_frags_loading<0, 4, 1, 0, 12>(acc, f0, f1, tiles_u32 + s * STAGE_BYTES, lm);
        if (more) {
          if (!ready && !wait_bounded_inline(full_bar + 8 * s1, ph1, abort_flag, p)) { ok = false; break; }
          mma_frags_loading<0, 2, 0, 0, 6>(acc, f1, f0, tiles_u32 + s1 * STAGE_BYTES, lm);
          release_stage(empty_bar + 8 * s, lane);
          mma_frags_loading<2, 4, 0, 6, 12>(acc, f1, f0, tiles_u32 + s1 * STAGE_BYTES, lm);
        } else {
          mma_frags<0, 2>(acc, f1);
          release_stage(empty_bar + 8 * s, lane);
          have = get_work(p, cta, nctas, idx + 1, wn);
          mma_frags<2, 4>(acc, f1);
        }
      }
      if (!ok) break;
      if (w.slot >= 0 || w.tn * BN + BN > p.N) {
        // a partial tile goes straight to the workspace; a tile of a ragged last tile column is added
        // to C by these warps themselves (the copy engine's untiled requests cannot clip a row)
        store_tile<WS_EPI_BATCH, 4, false>(p, w, lm, acc);
        continue;
      }
      // ---- the tile leaves through the copy engine
      // this slab's turn: the previous user's data (the other slab's) has been read by the copy engine.
      // Slab 0 starts; turn number `turns` of a slab is phase `turns` of its barrier (slab 0: turns - 1).
      // (the decision to leave is taken by the whole warp: once per tile, a vote is cheap)
      if (use > 0 && !__all_sync(0xffffffffu, wait_bounded_inline(c_turn + 8 * slab, ((use - 1) >> 1) & 1u, abort_flag, p) ? 1 : 0)) { ok = false; break; }
      if (p.alpha != 1.0) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
#pragma unroll
          for (int nt = 0; nt < 4; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] *= p.alpha;
      }
#pragma unroll
      for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int half = 0; half < 2; ++half)
#pragma unroll
          for (int np = 0; np < 2; ++np) {
            // first piece: columns 4t, 4t+1; second: columns 4t+2, 4t+3
            const double lo0 = acc[mt][2 * np][2 * half], lo1 = acc[mt][2 * np + 1][2 * half];
            const double hi0 = acc[mt][2 * np][2 * half + 1], hi1 = acc[mt][2 * np + 1][2 * half + 1];
            const uint32_t row = c_lane + (uint32_t)np * 128u + (uint32_t)((16 * mt + 8 * half) * WsBulkCfg::C_ROW_BYTES);
            ptx::sts128(row + ch_first, swap ? hi0 : lo0, swap ? hi1 : lo1);
            ptx::sts128(row + ch_second, swap ? lo0 : hi0, swap ? lo1 : hi1);
          }
      ptx::fence_proxy_async();  // these generic-proxy writes before the copy engine's reads
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(c_full);
      use += 2;
    }
  }
  ptx::named_barrier_sync(1, WsBulkCfg::THREADS_);  // all warps leave together
}

}  // namespace dgemm
