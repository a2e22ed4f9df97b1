// Host side of libdgemm: argument validation, variant choice, tensor-map creation and launch.
// Exports the C ABI declared in include/dgemm.h. Links only against the CUDA runtime; the one
// driver entry point needed (cuTensorMapEncodeTiled) is obtained through the runtime.
#include "../../include/dgemm.h"

#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "dgemm_dmma.cuh"
#include "dgemm_cluster.cuh"
#include "dgemm_bulk_epi.cuh"
#include "scratch_pool.h"

namespace {

using namespace dgemm;

constexpr int kMaxDevices = 64;
constexpr size_t kWorkspaceBytes = 640ull * BM * BN * sizeof(double);  // 80 MiB: up to 640 partial-tile slots
constexpr unsigned long long kWaitLimitNs = 4000000000ull;            // 4 s per device-side wait
constexpr int kAutoGeneric = DGEMM_VARIANT_GENERIC;  // what DGEMM_VARIANT_AUTO picks for operands TMA cannot address
// Tile columns of 32 (the 256 x 32 tile, about 83 % of the pipe) against tile columns of 128 (about
// 97 %): the narrow tile wins when its padded width, weighted by that ratio, is the smaller one
// (measured 8192 x 64 x 8192: 489 -> 275 us). Not beyond N = 96: the A panel is re-read from L2 once
// per tile column, and with five columns (6514 x 146 x 4725) that traffic, not the pipe, sets the pace.
// Tile columns of 64 (128 x 64 tiles, two CTAs per SM, the same warp tiles and bytes per flop as the
// 64 x 128 tile) when that saves at least a tenth of the padded width: N mod 128 in 1..64 for N up to ~700.
inline bool half_width_tiles_pay(int64_t N) {
  const int64_t cols64 = (N + 63) / 64 * 64, cols128 = (N + 127) / 128 * 128;
  return (double)cols64 * 1.10 <= (double)cols128;
}

// 256 x 32 tiles for a narrow N: when they cover clearly less padded area than 64 x 128 tiles would
// (in N alone for a tall problem; a short M turns the comparison around: 64 x 64 x 262144 ran 273 us
// on one 256 x 64 strip pair and 75 % padding, against 163 us for cuBLAS)
inline bool narrow_tiles_pay(int64_t M, int64_t N) {
  const int64_t cols32 = (N + 31) / 32 * 32, cols128 = (N + 127) / 128 * 128;
  const int64_t rows256 = (M + 255) / 256 * 256, rows64 = (M + 63) / 64 * 64;
  return N <= 96 && (double)rows256 * (double)cols32 * 1.2 < (double)rows64 * (double)cols128;
}
constexpr int kAutoWs64MaxKblocksPerCta = 256;     // ... and its 64-row form instead of the inline kernel up to this much work
constexpr int kAutoBulkMaxKblocks = 128;            // bulk-epilogue kernel: up to this many k-blocks per tile (K <= 2048: against the
                                                     // warp-specialised kernels 16 % faster at K = 64, 9 % at 128 ... 256, 1 % at 1024,
                                                     // 0.4 % at 2048, level at 4096) ...
constexpr int kAutoBulkMinWaves = 2;                 // ... and from this many waves of 128 x 128 tiles (2.2 ... 3.9 waves: 3 - 15 %
                                                     // faster; 1.7 waves: 4 % slower at K = 64)
constexpr int kAutoWsMinKblocks = 16;                // warp-specialised kernel: 128-row tiles from K = 256 up, 64-row below
constexpr double kPackMinFlopPerByte = 32.0;      // pack unaligned operands only if the copy is this cheap
constexpr double kPackMinFlopPerByteNarrow = 8.0; // ... or this cheap where the generic staging would run the 256 x 32 tile, its slowest form
constexpr double kPackMinFlop = 0.25e9;            // ... and the problem is not one of a few microseconds, where one more launch shows
constexpr double kPackMinElemsOfC = 8.0e6;         // (a large C with a tiny K is not one either: the pass over C alone takes 20 us and more)
constexpr size_t kPackMaxBytes = 2ull << 30;       // ... and the packed copies fit in 2 GiB
constexpr int64_t kHostBlockRows = 1024;             // dgemm_f64_host: rows of A and C per pipelined block
constexpr int64_t kHostPanelRows = 1024;             // ... and rows of B per panel while the first blocks wait for B
constexpr int kHostMaxBufs = 5;                      // ... and device buffers for blocks of A and C (3 first blocks + a ring of 2)
constexpr int kTailMinSpan = 1;          // stream-K tail: at least this many k-blocks per CTA
constexpr double kTailMinSavedKblocks = 5.0;  // use the stream-K tail only if it saves this many k-block times
// Cluster split-K (one launch, reduction through distributed shared memory) replaces the workspace
// split on a problem of less than one wave when its critical path, in k-blocks of a 64 x 128 tile
// (about 1 us each on an SM of its own), is at most this much longer: what the second launch and
// the workspace round trip cost.
constexpr int kClusterCreditKblocks = 1;
constexpr int kClusterMaxKblocks = 8;
// Column split of a ragged N (launch_gemm): M * K * (columns of arithmetic saved) above which the second launch pays
constexpr double kColumnSplitMinWork = 2.0e8;
constexpr double kColumnSplitMinWorkNarrow = 8.0e8;  // ... for N below 1024

// Whether a product with N columns is run as two products on a column split (launch_gemm): the
// shape part of the rule; the caller adds what depends on the operands and the settings.
inline bool column_split_shape(int64_t M, int64_t N, int64_t K) {
  const int64_t r = N % 128, r32 = (r + 31) / 32 * 32;
  const bool wide = N >= 1024;  // below, 128 x 64 tiles are the alternative and only a remainder of one 32-column strip pays
  return N > 128 && r >= 1 && r <= (wide ? 64 : 32) &&
         (double)M * (double)K * (128.0 - 1.2 * (double)r32) > (wide ? kColumnSplitMinWork : kColumnSplitMinWorkNarrow);
}

__device__ int g_status_word;  // one per device that loads the library

struct DeviceState {
  bool ready = false;
  int sm_count = 0;
  bool two_ctas_ok = false;    // the 64-row kernels fit two CTAs per SM on this device
  bool ws_ok[4] = {false, false, false, false};  // register pool of the warp-specialised kernels checked: TMA 128, generic 128, TMA 64, bulk epilogue
  bool cluster_ok = false;     // a cluster of 8 CTAs of the cluster split-K kernel can be resident
  bool bt_ok = false;          // register pool of the warp-specialised kernels that stage a transposed B checked
  int* status = nullptr;       // device address of g_status_word
  scratch::Pool scratch;       // split-K partial tiles and packed operand copies, leased per call (scratch_pool.h)
  cudaMemPool_t host_pool = nullptr;  // dgemm_f64_host: device copies of the operands come from this pool
};

DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;
std::atomic<int> g_variant{DGEMM_VARIANT_AUTO};
std::atomic<int> g_split_k{0};
std::atomic<int> g_test_flags{0};
std::atomic<long long> g_launches{0};
std::atomic<long long> g_test_wait_limit_ns{0};  // 0: the default limit of the device-side waits

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

// Launch with programmatic stream serialization: the grid may be scheduled while the kernel before
// it in the stream is draining; every kernel launched this way executes griddepcontrol.wait before
// its first access to global memory, which returns once that earlier kernel has completed and
// its writes are visible. Hides a few microseconds of launch latency per kernel.
template <typename... KArgs, typename... Args>
void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Launch of `grid` CTAs in clusters of `cluster` consecutive CTAs, with programmatic stream
// serialization as above.
template <typename... KArgs, typename... Args>
void launch_cluster_pdl(void (*kernel)(KArgs...), int grid, int cluster, int threads, size_t smem, cudaStream_t stream,
                        Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(threads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <typename Kernel>
void launch_gemm_kernel(Kernel kernel, int grid, int threads, int smem, cudaStream_t stream, const CUtensorMap& map_a,
                        const CUtensorMap& map_b, const GemmParams& p) {
  launch_pdl(kernel, dim3(grid), dim3(threads), (size_t)smem, stream, map_a, map_b, p);
}

template <bool USE_TMA, int TBM, int WTM, int TBN = BN>
void launch_tile_kernel(int grid, cudaStream_t stream, const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmParams& p) {
  launch_gemm_kernel(dgemm_dmma_kernel<USE_TMA, TBM, WTM, TBN>, grid, TileCfg<TBM, WTM, TBN>::THREADS_,
                     TileCfg<TBM, WTM, TBN>::SMEM_BYTES_, stream, map_a, map_b, p);
}

template <bool USE_TMA>
void launch_dfma_kernel(int grid, cudaStream_t stream, const CUtensorMap& map_a, const CUtensorMap& map_b, const GemmParams& p) {
  launch_gemm_kernel(dgemm_dmma_kernel<USE_TMA, 64, 64, BN, MICRO_DFMA>, grid, TileCfg<64, 64, BN>::THREADS_,
                     TileCfg<64, 64, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
}

template <bool USE_TMA>
void launch_default_kernel(int bm, int wtm, int grid, cudaStream_t stream, const CUtensorMap& map_a,
                           const CUtensorMap& map_b, const GemmParams& p) {
  if (p.bn == 64) launch_tile_kernel<USE_TMA, 128, 64, 64>(grid, stream, map_a, map_b, p);
  else if (bm == 256) launch_tile_kernel<USE_TMA, 256, 64, 32>(grid, stream, map_a, map_b, p);
  else if (bm == 32) launch_tile_kernel<USE_TMA, 32, 32>(grid, stream, map_a, map_b, p);
  else if (bm == 128 && wtm == 64) launch_tile_kernel<USE_TMA, 128, 64>(grid, stream, map_a, map_b, p);
  else if (bm == 128) launch_tile_kernel<USE_TMA, 128, 32>(grid, stream, map_a, map_b, p);
  else if (wtm == 64) launch_tile_kernel<USE_TMA, 64, 64>(grid, stream, map_a, map_b, p);
  else launch_tile_kernel<USE_TMA, 64, 32>(grid, stream, map_a, map_b, p);
}

template <bool USE_TMA, int TBM, int WTM, int TBN = BN, int MICRO = MICRO_DMMA>
bool configure_tile_kernel(int* occupancy) {
  auto* k = dgemm_dmma_kernel<USE_TMA, TBM, WTM, TBN, MICRO>;
  if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<TBM, WTM, TBN>::SMEM_BYTES_) != cudaSuccess) return false;
  if (cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) return false;
  return cudaOccupancyMaxActiveBlocksPerMultiprocessor(occupancy, k, TileCfg<TBM, WTM, TBN>::THREADS_,
                                                       TileCfg<TBM, WTM, TBN>::SMEM_BYTES_) == cudaSuccess;
}

// Shared-memory opt-in of the instantiations that stage transposed operands themselves.
template <int TBM, int WTM, int TBN, bool BT, bool AT>
bool configure_transposed_tile() {
  auto* k = dgemm_dmma_kernel<true, TBM, WTM, TBN, MICRO_DMMA, BT, AT>;
  return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<TBM, WTM, TBN>::SMEM_BYTES_) == cudaSuccess &&
         cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess;
}

template <bool BT, bool AT>
bool configure_transposed_kernels() {
  return cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true, 128, BT, AT>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true, 64, BT, AT>, cudaFuncAttributeMaxDynamicSharedMemorySize, WsCfg<64>::SMEM_BYTES_) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true, 64, BT, AT>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_dmma_kernel<true, 64, 64, BN, MICRO_DMMA, BT, AT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TileCfg<64, 64, BN>::SMEM_BYTES_) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_dmma_kernel<true, 64, 64, BN, MICRO_DMMA, BT, AT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxShared) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_cluster_kernel<true, 64, 64, BN, BT, AT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              TileCfg<64, 64, BN>::SMEM_BYTES_) == cudaSuccess &&
         cudaFuncSetAttribute(dgemm_cluster_kernel<true, 64, 64, BN, BT, AT>, cudaFuncAttributePreferredSharedMemoryCarveout,
                              cudaSharedmemCarveoutMaxShared) == cudaSuccess &&
         configure_transposed_tile<128, 64, 64, BT, AT>() && configure_transposed_tile<256, 64, 32, BT, AT>() &&
         configure_transposed_tile<32, 32, BN, BT, AT>();
}

// Per-device set-up, once: capability check, SM count, status-word address, shared-memory opt-in.
int device_state(DeviceState** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return DGEMM_ERR_DEVICE;
  }
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState& st = g_dev[dev];
  if (!st.ready) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      (void)cudaGetLastError();
      return DGEMM_ERR_DEVICE;
    }
    if (major != 10) return DGEMM_ERR_DEVICE;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&st.status), g_status_word) != cudaSuccess) return DGEMM_ERR_CUDA;
    if (cudaMemset(st.status, 0, sizeof(int)) != cudaSuccess) return DGEMM_ERR_CUDA;
    int occ[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    const bool attr_ok =
        configure_tile_kernel<true, 128, 64, 64>(&occ[12]) && configure_tile_kernel<false, 128, 64, 64>(&occ[13]) &&
        configure_tile_kernel<true, 32, 32>(&occ[10]) && configure_tile_kernel<false, 32, 32>(&occ[11]) &&
        configure_tile_kernel<true, 128, 64>(&occ[0]) && configure_tile_kernel<false, 128, 64>(&occ[1]) &&
        configure_tile_kernel<true, 128, 32>(&occ[2]) && configure_tile_kernel<false, 128, 32>(&occ[3]) &&
        configure_tile_kernel<true, 64, 64>(&occ[4]) && configure_tile_kernel<false, 64, 64>(&occ[5]) &&
        configure_tile_kernel<true, 64, 32>(&occ[6]) && configure_tile_kernel<false, 64, 32>(&occ[7]) &&
        configure_tile_kernel<true, 256, 64, 32>(&occ[8]) && configure_tile_kernel<false, 256, 64, 32>(&occ[9]) &&
        configure_tile_kernel<true, 64, 64, BN, MICRO_DFMA>(&occ[14]) && configure_tile_kernel<false, 64, 64, BN, MICRO_DFMA>(&occ[15]) &&
        cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(dgemm_dmma_ws_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true, 64>, cudaFuncAttributeMaxDynamicSharedMemorySize, WsCfg<64>::SMEM_BYTES_) == cudaSuccess &&
        cudaFuncSetAttribute(dgemm_dmma_ws_kernel<true, 64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess &&
        configure_transposed_kernels<true, false>() && configure_transposed_kernels<false, true>() && configure_transposed_kernels<true, true>();
    if (!attr_ok) return DGEMM_ERR_CUDA;
    // the 64-row kernels are meant to run two CTAs per SM; use them only where the device really fits two
    st.two_ctas_ok = occ[4] >= 2 && occ[5] >= 2 && occ[6] >= 2 && occ[7] >= 2 && occ[8] >= 2 && occ[9] >= 2 && occ[10] >= 2 && occ[11] >= 2 && occ[12] >= 2 && occ[13] >= 2 && occ[14] >= 2 && occ[15] >= 2;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
          qres != cudaDriverEntryPointSuccess || !fn)
        return DGEMM_ERR_CUDA;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    // setmaxnreg moves registers inside the pool the CTA owns at launch (threads x registers per
    // thread as compiled); a consumer warpgroup asking for more than the pool holds would wait for
    // ever. Check the arithmetic against what the compiler actually allocated before using them.
    {
      cudaFuncAttributes fa;
      auto pool_ok = [&](const void* fn, int threads, int consumer_threads, int producer_regs) {
        if (cudaFuncGetAttributes(&fa, fn) != cudaSuccess) {
          (void)cudaGetLastError();
          return false;
        }
        return fa.numRegs * threads >= consumer_threads * WS_CONSUMER_REGS + (threads - consumer_threads) * producer_regs;
      };
      st.ws_ok[0] = pool_ok(reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 128>), WsCfg<128>::THREADS_,
                            WsCfg<128>::CONSUMER_WARPS * 32, WsCfg<128>::PRODUCER_REGS);
      st.ws_ok[1] = pool_ok(reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<false, 128>), WsCfg<128>::THREADS_,
                            WsCfg<128>::CONSUMER_WARPS * 32, WsCfg<128>::PRODUCER_REGS);
      st.ws_ok[2] = pool_ok(reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 64>), WsCfg<64>::THREADS_,
                            WsCfg<64>::CONSUMER_WARPS * 32, WsCfg<64>::PRODUCER_REGS);
      st.bt_ok = true;  // (bt_ok: every instantiation that stages a transposed operand has its register pool)
      {
        const void* k128[3] = {reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 128, true, false>),
                               reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 128, false, true>),
                               reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 128, true, true>)};
        const void* k64[3] = {reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 64, true, false>),
                              reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 64, false, true>),
                              reinterpret_cast<const void*>(dgemm_dmma_ws_kernel<true, 64, true, true>)};
        for (int i = 0; i < 3; ++i)
          st.bt_ok = st.bt_ok && pool_ok(k128[i], WsCfg<128>::THREADS_, WsCfg<128>::CONSUMER_WARPS * 32, WsCfg<128>::PRODUCER_REGS) &&
                     pool_ok(k64[i], WsCfg<64>::THREADS_, WsCfg<64>::CONSUMER_WARPS * 32, WsCfg<64>::PRODUCER_REGS);
      }
      st.ws_ok[3] = cudaFuncSetAttribute(dgemm_dmma_wsb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         WsBulkCfg::SMEM_BYTES_) == cudaSuccess &&
                    pool_ok(reinterpret_cast<const void*>(dgemm_dmma_wsb_kernel), WsBulkCfg::THREADS_,
                            WsBulkCfg::CONSUMER_WARPS * 32, WS_PRODUCER_REGS);
      (void)cudaGetLastError();
    }
    {
      // cluster split-K kernel: shared-memory opt-in, then ask whether a full-size cluster fits
      auto* ck = dgemm_cluster_kernel<true, 64, 64, BN>;
      auto* ckg = dgemm_cluster_kernel<false, 64, 64, BN>;
      using CCfg = TileCfg<64, 64, BN>;
      st.cluster_ok = false;
      if (cudaFuncSetAttribute(ck, cudaFuncAttributeMaxDynamicSharedMemorySize, CCfg::SMEM_BYTES_) == cudaSuccess &&
          cudaFuncSetAttribute(ck, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess &&
          cudaFuncSetAttribute(ckg, cudaFuncAttributeMaxDynamicSharedMemorySize, CCfg::SMEM_BYTES_) == cudaSuccess &&
          cudaFuncSetAttribute(ckg, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(CLUSTER_MAX);
        cfg.blockDim = dim3(CCfg::THREADS_);
        cfg.dynamicSmemBytes = CCfg::SMEM_BYTES_;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = CLUSTER_MAX;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        int clusters_g = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, ck, &cfg) == cudaSuccess &&
            cudaOccupancyMaxActiveClusters(&clusters_g, ckg, &cfg) == cudaSuccess)
          st.cluster_ok = clusters >= 1 && clusters_g >= 1;
      }
      (void)cudaGetLastError();
    }
    st.sm_count = sms;
    st.ready = true;
  }
  *out = &st;
  return DGEMM_OK;
}

// Memory pool of dgemm_f64_host. The device's default pool gives memory back to the system at
// every synchronisation, so each call would pay for mapping its 0.8 GB (8192^3) again: more than
// the copies and the arithmetic together. This pool keeps up to kHostPoolKeepBytes between calls.
constexpr unsigned long long kHostPoolKeepBytes = 6ull << 28;  // 1.5 GiB: B, five blocks of A and C and three more of C at 8192^3 (1.31 GiB)
int ensure_host_pool(DeviceState* st, cudaMemPool_t* pool) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!st->host_pool) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DGEMM_ERR_DEVICE;
    cudaMemPoolProps props;
    memset(&props, 0, sizeof(props));
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = dev;
    cudaMemPool_t created = nullptr;
    unsigned long long keep = kHostPoolKeepBytes;
    if (cudaMemPoolCreate(&created, &props) == cudaSuccess &&
        cudaMemPoolSetAttribute(created, cudaMemPoolAttrReleaseThreshold, &keep) == cudaSuccess) {
      st->host_pool = created;
    } else {
      // no pool of our own (an unusual driver configuration): the device's default pool still
      // works, only slower, as it keeps nothing between calls
      (void)cudaGetLastError();
      if (created) cudaMemPoolDestroy(created);
      cudaMemPool_t fallback = nullptr;
      if (cudaDeviceGetDefaultMemPool(&fallback, dev) != cudaSuccess || !fallback) {
        (void)cudaGetLastError();
        return DGEMM_ERR_CUDA;
      }
      *pool = fallback;
      return DGEMM_OK;
    }
  }
  *pool = st->host_pool;
  return DGEMM_OK;
}

// 2-D f64 tensor map: inner extent `cols` (contiguous), outer extent `rows` with stride ld
// doubles; box = box_cols x box_rows; 128-byte swizzle; out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const double* base, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(double)};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<double*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view of a row-major K x N matrix whose N is a multiple of 16: (column within a block of 16,
// k, block of 16 columns), box 16 x box_k x box_blocks. One copy then lands as `box_blocks`
// consecutive [box_k][16] sub-tiles, each row 128 bytes, 128-byte swizzled: the B stage layout.
bool make_blocked_map(CUtensorMap* map, const double* base, int64_t K, int64_t N, int64_t ld, int box_k, int box_blocks) {
  const cuuint64_t dims[3] = {16, (cuuint64_t)K, (cuuint64_t)(N / 16)};
  const cuuint64_t strides[2] = {(cuuint64_t)ld * sizeof(double), 16 * sizeof(double)};
  const cuuint32_t box[3] = {16, (cuuint32_t)box_k, (cuuint32_t)box_blocks};
  const cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 3, const_cast<double*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool ranges_overlap(const void* p, int64_t pbytes, const void* q, int64_t qbytes) {
  const uintptr_t a = (uintptr_t)p, b = (uintptr_t)q;
  return a < b + (uintptr_t)qbytes && b < a + (uintptr_t)pbytes;
}

// Everything that can be decided without touching the device. Returns 1 for "nothing to do".
// A is stored (ta ? K x M : M x K), B is stored (tb ? N x K : K x N). `scales_c`: the call may
// have to rewrite C even without a product (general form with beta != 1); then K == 0 or
// `no_product` (alpha == 0) returns 2 after checking C alone, A and B stay unexamined.
int validate(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
             const double* C, int64_t ldc, bool ta = false, bool tb = false, bool scales_c = false,
             bool no_product = false) {
  const int64_t kMaxDim = (int64_t)INT32_MAX - 2 * BM;
  if (M < 0 || N < 0 || K < 0 || M > kMaxDim || N > kMaxDim || K > kMaxDim) return DGEMM_ERR_BAD_DIM;
  if (M == 0 || N == 0) return 1;
  const int64_t a_rows = ta ? K : M, a_cols = ta ? M : K, b_rows = tb ? N : K, b_cols = tb ? K : N;
  if (lda < (a_cols > 0 ? a_cols : 1) || ldb < (b_cols > 0 ? b_cols : 1) || ldc < N) return DGEMM_ERR_BAD_LD;
  if (K == 0 || no_product) {
    if (!scales_c) return 1;
    if (!C) return DGEMM_ERR_NULL;
    if ((uintptr_t)C & 7) return DGEMM_ERR_ALIGN;
    return 2;
  }
  if (!A || !B || !C) return DGEMM_ERR_NULL;
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 7) return DGEMM_ERR_ALIGN;
  const int64_t abytes = ((a_rows - 1) * lda + a_cols) * 8, bbytes = ((b_rows - 1) * ldb + b_cols) * 8,
                cbytes = ((M - 1) * ldc + N) * 8;
  if (ranges_overlap(C, cbytes, A, abytes) || ranges_overlap(C, cbytes, B, bbytes)) return DGEMM_ERR_ALIAS;
  const int64_t tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  if (tiles > (int64_t)INT32_MAX / 512) return DGEMM_ERR_BAD_DIM;
  return DGEMM_OK;
}

inline unsigned grid_y(int64_t blocks) { return (unsigned)(blocks < 65535 ? blocks : 65535); }

// Everything launch_gemm decides from the shape alone: which kernel, which tile, how the work is
// cut. A pure function of its arguments (no device, no globals), so that it can be tested on a
// machine without a GPU through dgemm_plan().
struct Plan {
  int status;        // DGEMM_OK, or the error the call would return
  int variant;       // resolved DGEMM_VARIANT_* (never AUTO)
  int bm, bn;        // CTA tile
  int wtm;           // rows of a warp tile (64 or 32)
  int ctas_per_sm;
  int grid;          // CTAs launched (all resident at once)
  int kblocks;       // ceil(K / 16)
  int split_k, kblocks_per_split;       // phase 1: uniform K split (1 unless forced)
  int dp_tiles, tail_tiles, tail_ipc;   // whole tiles / tiles of the last partial wave / k-blocks per CTA span
};

// The cluster split-K kernel on `tiles` 64 x 128 tiles with clusters of s CTAs.
void fill_cluster_plan(Plan& pl, int tiles, int kblocks, int s, bool tma) {
  pl.variant = tma ? DGEMM_VARIANT_TMA_CLUSTER : DGEMM_VARIANT_GENERIC_CLUSTER;
  pl.bm = 64;
  pl.bn = BN;
  pl.wtm = 64;
  pl.ctas_per_sm = 2;
  pl.grid = tiles * s;
  pl.split_k = s;
  pl.kblocks_per_split = (kblocks + s - 1) / s;
  pl.dp_tiles = tiles;
  pl.tail_tiles = 0;
  pl.tail_ipc = 1;
}

Plan plan_gemm(int64_t M, int64_t N, int64_t K, bool tma_ok, int requested_variant, int dbg_flags, int forced_split,
               int sm_count, bool two_ctas_ok, const bool ws_ok[4], bool cluster_ok, bool c_bulk_ok) {
  Plan pl;
  memset(&pl, 0, sizeof(pl));
  pl.status = DGEMM_OK;
  int variant = requested_variant;
  const bool auto_choice = requested_variant == DGEMM_VARIANT_AUTO;
  const int kblocks = (int)((K + BK - 1) / BK);
  pl.kblocks = kblocks;
  bool auto_ws64 = false;  // AUTO wants the warp-specialised kernel in its 64-row form although K >= 256
  if (auto_choice) {
    if (!tma_ok) {
      variant = kAutoGeneric;
    } else {
      // The warp-specialised kernel (128 x 128 tiles, one CTA per SM, software-pipelined consumers)
      // has the fastest main loop. The inline kernel with 64-row tiles and two CTAs per SM wastes
      // less on an M just above a multiple of 64, and has the narrow, half-width and short tiles.
      // For K < 256 the warp-specialised kernel itself runs 64-row tiles, two CTAs per SM (below).
      const int64_t pad128 = (M + 127) / 128 * 128, pad64 = (M + 63) / 64 * 64;
      const bool short_k = kblocks < kAutoWsMinKblocks;
      const int64_t tiles128 = (pad128 / 128) * ((N + BN - 1) / BN);
      // (a handful of tiles: the inline kernel starts faster, 14 against 18 us at 256^3)
      const bool short_rows = M <= 512 && (M + 31) / 32 * 32 < pad64;  // 32-row tiles of the inline kernel, below
      const bool std_tile = !narrow_tiles_pay(M, N) && !half_width_tiles_pay(N) && !short_rows;
      const bool ws = std_tile && tiles128 >= 16 && (short_k || (double)pad128 <= 1.03 * (double)pad64);
      // Where 64-row tiles are the better fit, the warp-specialised kernel's 64-row form beats the
      // inline kernel on problems of up to a few hundred microseconds (26 random shapes: 4 % in the
      // geometric mean, up to 11 %; its producer warps keep the stages full across the short tiles'
      // epilogues), and loses up to 0.8 % on long ones: taken up to 256 k-blocks per resident CTA.
      if (!ws && std_tile && two_ctas_ok && ws_ok[2]) {
        const int64_t tiles64 = (pad64 / 64) * ((N + BN - 1) / BN);
        auto_ws64 = tiles64 * kblocks <= (int64_t)kAutoWs64MaxKblocksPerCta * 2 * sm_count;
      }
      variant = ((ws && ws_ok[0] && ws_ok[2]) || auto_ws64) ? DGEMM_VARIANT_TMA_WS : DGEMM_VARIANT_TMA;
      // Many tiles of few k-blocks each (a rank-k update): the C round trip of a tile is long next to
      // its arithmetic. The bulk-epilogue kernel takes it off the arithmetic warps altogether.
      if (std_tile && c_bulk_ok && ws_ok[3] && kblocks <= kAutoBulkMaxKblocks && tiles128 >= (int64_t)kAutoBulkMinWaves * sm_count &&
          (double)pad128 <= 1.03 * (double)pad64 && !(dbg_flags & DGEMM_TEST_WS_TWO_CTAS))
        variant = DGEMM_VARIANT_TMA_WS_BULK;
    }
  }
  pl.variant = variant;
  const bool dfma = variant == DGEMM_VARIANT_TMA_DFMA || variant == DGEMM_VARIANT_GENERIC_DFMA;
  const bool wants_tma = variant == DGEMM_VARIANT_TMA || variant == DGEMM_VARIANT_TMA_WS || variant == DGEMM_VARIANT_TMA_CLUSTER ||
                         variant == DGEMM_VARIANT_TMA_DFMA || variant == DGEMM_VARIANT_TMA_WS_BULK;
  if (wants_tma && !tma_ok) { pl.status = DGEMM_ERR_VARIANT; return pl; }
  if (variant == DGEMM_VARIANT_TMA_WS_BULK && !(c_bulk_ok && ws_ok[3])) { pl.status = DGEMM_ERR_VARIANT; return pl; }
  if (dfma && !two_ctas_ok) { pl.status = DGEMM_ERR_VARIANT; return pl; }
  if (variant == DGEMM_VARIANT_TMA_CLUSTER || variant == DGEMM_VARIANT_GENERIC_CLUSTER) {
    // forced: clusters of dgemm_set_split_k() CTAs if that is 1, 2, 4 or 8 (ranks beyond the last
    // k-block then idle), else the largest size that keeps all CTAs resident at once
    if (!cluster_ok || !two_ctas_ok) { pl.status = DGEMM_ERR_VARIANT; return pl; }
    const int64_t tiles64 = ((M + 63) / 64) * ((N + BN - 1) / BN);
    if (tiles64 > (int64_t)INT32_MAX / 16) { pl.status = DGEMM_ERR_BAD_DIM; return pl; }
    int s = 1;
    if (forced_split == 1 || forced_split == 2 || forced_split == 4 || forced_split == 8) {
      s = forced_split;
    } else {
      while (s < CLUSTER_MAX && 2 * s <= kblocks && tiles64 * 2 * s <= 2 * (int64_t)sm_count) s *= 2;
    }
    fill_cluster_plan(pl, (int)tiles64, kblocks, s, variant == DGEMM_VARIANT_TMA_CLUSTER);
    return pl;
  }
  if ((variant == DGEMM_VARIANT_TMA_WS && !(ws_ok[0] && ws_ok[2])) || (variant == DGEMM_VARIANT_GENERIC_WS && !ws_ok[1])) {
    pl.status = DGEMM_ERR_VARIANT;
    return pl;
  }
  if (variant == DGEMM_VARIANT_NAIVE || variant == DGEMM_VARIANT_SMEM) {
    pl.bm = variant == DGEMM_VARIANT_NAIVE ? 8 : SMEM_RUNG_TILE;
    pl.bn = 32; pl.wtm = 0; pl.ctas_per_sm = 0;
    pl.grid = 0; pl.split_k = 1; pl.kblocks_per_split = kblocks;
    return pl;
  }

  const bool ws_variant = variant == DGEMM_VARIANT_TMA_WS || variant == DGEMM_VARIANT_GENERIC_WS || variant == DGEMM_VARIANT_TMA_WS_BULK;
  // tile height of the chosen kernel: 64 rows with two CTAs per SM (inline kernel; warp-specialised kernel for short K),
  // 128 rows with one CTA per SM (warp-specialised kernel otherwise, large generic problems, test flag)
  // (generic staging on a problem of many waves is a little faster with the tall tile: half the B copies per thread)
  const int64_t tiles128 = ((M + 127) / 128) * ((N + BN - 1) / BN);
  const bool generic_large = !wants_tma && tiles128 >= 4 * (int64_t)sm_count;
  // (the micro-kernel swap exists for the 64 x 128 tile only and ignores the tile-shape flags)
  const bool plain_tiles = dfma || (dbg_flags & (DGEMM_TEST_TALL_TILES | DGEMM_TEST_SMALL_WARP_TILES)) != 0;
  // narrow problems (see narrow_tiles_pay) use 256 x 32 tiles: four warps stacked in M, little arithmetic on unused columns
  const bool narrow = narrow_tiles_pay(M, N) && !ws_variant && !plain_tiles && two_ctas_ok;
  // N just above a multiple of 128: 128 x 64 tiles
  const bool half_width = auto_choice && !ws_variant && !narrow && half_width_tiles_pay(N) && two_ctas_ok && !plain_tiles;
  // short problems in M (M <= 32, or a last 64-row tile that is at most half full while M is small) use 32 x 128
  // tiles of four 32 x 32 warp tiles: no arithmetic on unused rows
  const int64_t pad32 = (M + 31) / 32 * 32, pad64m = (M + 63) / 64 * 64;
  const bool short_m = auto_choice && !ws_variant && !narrow && !half_width && M <= 512 && pad32 < pad64m && two_ctas_ok &&
                       !plain_tiles && !(dbg_flags & DGEMM_TEST_WS_TWO_CTAS);
  // warp-specialised with 64-row tiles, two CTAs per SM: the second CTA hides the C round trip of short-K problems
  const bool ws64 = variant == DGEMM_VARIANT_TMA_WS && two_ctas_ok &&
                    (kblocks < kAutoWsMinKblocks || auto_ws64 || (dbg_flags & DGEMM_TEST_WS_TWO_CTAS));
  const int bm = narrow ? 256 : half_width ? 128 : short_m ? 32 : (ws64 || dfma) ? 64
                 : (ws_variant || generic_large || (dbg_flags & DGEMM_TEST_TALL_TILES) || !two_ctas_ok) ? 128 : 64;
  const int bn = narrow ? 32 : half_width ? 64 : BN;
  pl.bm = bm;
  pl.bn = bn;
  pl.wtm = (short_m || (!dfma && (dbg_flags & DGEMM_TEST_SMALL_WARP_TILES))) ? 32 : 64;
  pl.ctas_per_sm = (bm == 128 && bn == 128) ? 1 : 2;

  const int64_t tiles64 = ((M + bm - 1) / bm) * ((N + bn - 1) / bn);
  if (tiles64 > (int64_t)INT32_MAX / 2) { pl.status = DGEMM_ERR_BAD_DIM; return pl; }
  const int tiles = (int)tiles64;
  const int sms = sm_count * pl.ctas_per_sm;  // concurrently resident CTAs
  const int max_partials = (int)(kWorkspaceBytes / (BM * BN * sizeof(double)));
  if (forced_split > 0) {
    // uniform split-K over all tiles (tests and ablation)
    int split = forced_split > kblocks ? kblocks : forced_split;
    if ((int64_t)split * tiles > max_partials) split = max_partials / tiles;
    if (split < 1) split = 1;
    pl.kblocks_per_split = (kblocks + split - 1) / split;
    pl.split_k = (kblocks + pl.kblocks_per_split - 1) / pl.kblocks_per_split;  // no empty partitions
    pl.dp_tiles = tiles;
    pl.tail_tiles = 0;
    pl.tail_ipc = 1;
    const int64_t units = (int64_t)tiles * pl.split_k;
    pl.grid = units < sms ? (int)units : sms;
  } else {
    // whole waves of tiles run data-parallel; the last partial wave is spread evenly over the SMs
    // (stream-K) when that saves more time than the partial-tile round trip costs
    pl.split_k = 1;
    pl.kblocks_per_split = kblocks;
    pl.dp_tiles = (tiles / sms) * sms;
    pl.tail_tiles = tiles - pl.dp_tiles;
    pl.tail_ipc = kblocks;
    pl.grid = tiles < sms ? tiles : sms;
    if (pl.tail_tiles > 0) {
      const double idle_kblocks = (1.0 - (double)pl.tail_tiles / sms) * kblocks;  // per-SM idle time if run as one wave
      if (idle_kblocks >= kTailMinSavedKblocks && kblocks >= 2 * kTailMinSpan &&
          (long long)(pl.tail_tiles + 1) * kblocks < (long long)INT32_MAX) {
        const long long total = (long long)pl.tail_tiles * kblocks;
        long long ipc = (total + sms - 1) / sms;
        if (ipc < kTailMinSpan) ipc = kTailMinSpan;
        if (ipc > kblocks) ipc = kblocks;
        pl.tail_ipc = (int)ipc;
        const int span_ctas = (int)((total + ipc - 1) / ipc);
        if (pl.dp_tiles == 0) pl.grid = span_ctas < sms ? span_ctas : sms;
      } else {
        pl.dp_tiles = tiles;  // run the last wave data-parallel as well
        pl.tail_tiles = 0;
      }
    }
    // Less than one wave of tiles: the cluster kernel cuts K over the CTAs of a cluster and adds the
    // partial tiles in shared memory, in one launch. Critical paths are compared in k-blocks of a
    // 64-row tile, doubled where two CTAs of the general kernels share an SM. Runs of more than 8
    // k-blocks per CTA stay with the general kernels, whose main loops are the faster ones. Any
    // test flag that asks for a particular tile or reduction keeps the general kernels too.
    if (auto_choice && cluster_ok && two_ctas_ok && !(dbg_flags & ~(DGEMM_TEST_NO_C_PREFETCH | DGEMM_TEST_NO_BLOCKED_B | DGEMM_TEST_DROP_LOADS)) && tiles < sms &&
        (pl.wtm == 64 || bm == 32)) {  // (not the test-only 32 x 32 warp tiles of the larger tiles)
      // costs in tenths of a k-block; a pass of the in-cluster reduction (512 element pairs per
      // CTA) is worth about 0.4 k-blocks, the second launch of the workspace split about one.
      // Only cluster sizes that leave every CTA an SM of its own: measured, clusters that have to
      // share SMs lose far more than the factor two of independent CTAs.
      const bool old_splits = pl.tail_tiles > 0 && pl.tail_ipc < kblocks;
      // (a k-block of a 32-row tile takes about half of a 64-row one; generic staging about 1.5 of TMA staging)
      const int path_old = (bm == 32 ? 5 : 10) * (old_splits ? pl.tail_ipc : kblocks) * ((bm == 128 || pl.grid > sm_count) ? 2 : 1) *
                           (wants_tma ? 2 : (bm == 256 ? 4 : 3)) / 2;  // (the 256 x 32 tile with generic staging: about 2)
      // (one k-block per CTA and the reduction kernel behind it is the general kernels' floor, 7.8 us
      // at 128^3, and below the cluster kernel's, 8.7 us: no credit there)
      const int cost_old = path_old + ((old_splits && path_old >= 20) ? 10 * kClusterCreditKblocks : 0);
      const int64_t tiles_c = ((M + 63) / 64) * ((N + BN - 1) / BN);
      int best_s = 0, best_cost = INT32_MAX;
      for (int s = 2; s <= CLUSTER_MAX; s *= 2) {  // (ranks beyond the last k-block still share in the reduction)
        const int kps = (kblocks + s - 1) / s;
        const int64_t alone = s >= 4 ? sm_count - sm_count / 8 : sm_count - 4;  // clusters are placed inside a GPC
        if (tiles_c * s > alone) break;
        if (kps > kClusterMaxKblocks) continue;
        const int cost = 10 * kps * (wants_tma ? 2 : 3) / 2 + 4 * (CLUSTER_MAX / s);
        if (cost < best_cost) { best_cost = cost; best_s = s; }
      }
      if (best_s > 0 && best_cost <= cost_old) fill_cluster_plan(pl, (int)tiles_c, kblocks, best_s, wants_tma);
    }
  }
  return pl;
}

// The scalars and operand forms of the general entry point; the defaults are the paper's C += A B.
struct GemmForm {
  bool ta = false, tb = false;  // A is stored K x M / B is stored N x K and used transposed
  double alpha = 1.0, beta = 1.0;
  bool native_bt = false;       // set by launch_gemm: B is still the stored N x K matrix and the kernel stages B^T itself
  bool native_at = false;       // likewise A is still the stored K x M matrix
};

// Kernels that can stage a transposed operand themselves (a tensor map over the matrix as stored): the
// warp-specialised kernels, the inline kernel's 64 x 128 tile and the cluster split-K kernel, all with TMA staging.
bool plan_supports_native_bt(const Plan& pl) {
  if (pl.status != DGEMM_OK) return false;
  if (pl.variant == DGEMM_VARIANT_TMA)  // the inline kernel's 64 x 128, 128 x 64, 256 x 32 and 32 x 128 tiles
    return (pl.bm == 64 && pl.bn == BN && pl.wtm == 64) || (pl.bm == 128 && pl.bn == 64 && pl.wtm == 64) ||
           (pl.bm == 256 && pl.bn == 32 && pl.wtm == 64) || (pl.bm == 32 && pl.bn == BN && pl.wtm == 32);
  if (pl.bn != BN || pl.wtm != 64) return false;
  if (pl.variant == DGEMM_VARIANT_TMA_WS) return pl.bm == 128 || pl.bm == 64;
  return pl.variant == DGEMM_VARIANT_TMA_CLUSTER && pl.bm == 64;
}

// The kernels that stage transposed operands themselves: 0 warp-specialised 128 x 128, 1 warp-specialised
// 64 x 128, 2 inline 64 x 128, 3 cluster split-K (64 x 128), 4 inline 128 x 64, 5 inline 256 x 32, 6 inline 32 x 128.
template <bool BT, bool AT>
void launch_transposed_kernel(int which, int grid, cudaStream_t stream, const CUtensorMap& map_a, const CUtensorMap& map_b,
                              const GemmParams& p) {
  if (which == 3)
    launch_cluster_pdl(dgemm_cluster_kernel<true, 64, 64, BN, BT, AT>, grid, p.split_k, TileCfg<64, 64, BN>::THREADS_,
                       (size_t)TileCfg<64, 64, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
  else if (which == 4)
    launch_gemm_kernel(dgemm_dmma_kernel<true, 128, 64, 64, MICRO_DMMA, BT, AT>, grid, TileCfg<128, 64, 64>::THREADS_,
                       TileCfg<128, 64, 64>::SMEM_BYTES_, stream, map_a, map_b, p);
  else if (which == 5)
    launch_gemm_kernel(dgemm_dmma_kernel<true, 256, 64, 32, MICRO_DMMA, BT, AT>, grid, TileCfg<256, 64, 32>::THREADS_,
                       TileCfg<256, 64, 32>::SMEM_BYTES_, stream, map_a, map_b, p);
  else if (which == 6)
    launch_gemm_kernel(dgemm_dmma_kernel<true, 32, 32, BN, MICRO_DMMA, BT, AT>, grid, TileCfg<32, 32, BN>::THREADS_,
                       TileCfg<32, 32, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
  else if (which == 0)
    launch_gemm_kernel(dgemm_dmma_ws_kernel<true, 128, BT, AT>, grid, WS_THREADS, SMEM_BYTES, stream, map_a, map_b, p);
  else if (which == 1)
    launch_gemm_kernel(dgemm_dmma_ws_kernel<true, 64, BT, AT>, grid, WsCfg<64>::THREADS_, WsCfg<64>::SMEM_BYTES_, stream, map_a, map_b, p);
  else
    launch_gemm_kernel(dgemm_dmma_kernel<true, 64, 64, BN, MICRO_DMMA, BT, AT>, grid, TileCfg<64, 64, BN>::THREADS_,
                       TileCfg<64, 64, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
}

// Plans and launches one product on operands that are final (packed or transposed already where
// that was needed): kernel choice, parameters, tensor maps, launches.
int launch_gemm_packed(DeviceState* st, scratch::Hold& hold, int variant, int64_t M, int64_t N, int64_t K, const double* A,
                       int64_t lda, const double* B, int64_t ldb, double* C, int64_t ldc, cudaStream_t stream,
                       const GemmForm& form) {
  int rc = DGEMM_OK;
  const bool tma_ok = (((uintptr_t)A | (uintptr_t)B) & 15) == 0 && (lda % 2 == 0) && (ldb % 2 == 0);
  const int dbg_flags = g_test_flags.load();
  // C as the copy engine needs it for the bulk epilogue, and a beta it can apply (add, or overwrite)
  const bool c_bulk_ok = !form.native_bt && !form.native_at && ((uintptr_t)C & 15) == 0 && (ldc % 2 == 0) && (form.beta == 1.0 || form.beta == 0.0);
  const Plan plan = plan_gemm(M, N, K, tma_ok, variant, dbg_flags, g_split_k.load(), st->sm_count, st->two_ctas_ok, st->ws_ok,
                              st->cluster_ok, c_bulk_ok);
  if (plan.status != DGEMM_OK) return plan.status;
  if ((form.native_bt || form.native_at) && !plan_supports_native_bt(plan)) return DGEMM_ERR_VARIANT;  // (launch_gemm asked the same plan first)
  variant = plan.variant;
  const bool dfma = variant == DGEMM_VARIANT_TMA_DFMA || variant == DGEMM_VARIANT_GENERIC_DFMA;
  const bool wants_tma = variant == DGEMM_VARIANT_TMA || variant == DGEMM_VARIANT_TMA_WS || variant == DGEMM_VARIANT_TMA_CLUSTER ||
                         variant == DGEMM_VARIANT_TMA_DFMA || variant == DGEMM_VARIANT_TMA_WS_BULK;
  const bool cluster = variant == DGEMM_VARIANT_TMA_CLUSTER || variant == DGEMM_VARIANT_GENERIC_CLUSTER;

  if (variant == DGEMM_VARIANT_NAIVE) {
    if (form.alpha != 1.0 || form.beta != 1.0) return DGEMM_ERR_VARIANT;  // the naive nest is C += A B only
    dim3 block(32, 8), grid((unsigned)((N + 31) / 32), (unsigned)((M + 7) / 8));
    dgemm_naive_kernel<<<grid, block, 0, stream>>>((int)M, (int)N, (int)K, A, lda, B, ldb, C, ldc);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? DGEMM_OK : DGEMM_ERR_CUDA;
  }
  if (variant == DGEMM_VARIANT_SMEM) {
    if (form.alpha != 1.0 || form.beta != 1.0) return DGEMM_ERR_VARIANT;  // a rung of the ladder: C += A B only
    dim3 block(SMEM_RUNG_TILE, SMEM_RUNG_TILE), grid((unsigned)((N + SMEM_RUNG_TILE - 1) / SMEM_RUNG_TILE),
                                                     grid_y((M + SMEM_RUNG_TILE - 1) / SMEM_RUNG_TILE));
    dgemm_smem_kernel<<<grid, block, 0, stream>>>((int)M, (int)N, (int)K, A, lda, B, ldb, C, ldc);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? DGEMM_OK : DGEMM_ERR_CUDA;
  }

  const int bm = plan.bm, bn = plan.bn, wtm = plan.wtm;
  const bool ws64 = variant == DGEMM_VARIANT_TMA_WS && bm == 64;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.bm = bm;
  p.bn = bn;
  p.tiles_m = (int)((M + bm - 1) / bm);
  p.tiles_n = (int)((N + bn - 1) / bn);
  p.A = A; p.B = B; p.C = C;
  p.lda = lda; p.ldb = ldb; p.ldc = ldc;
  {
    const long long test_limit = g_test_wait_limit_ns.load();
    p.wait_limit_ns = test_limit > 0 ? (unsigned long long)test_limit : kWaitLimitNs;
  }
  p.drop_loads = (dbg_flags & DGEMM_TEST_DROP_LOADS) ? 1 : 0;
  p.status = st->status;
  p.group_m = 1024 / bm;  // 1024 rows per raster group
  p.alpha = form.alpha;
  p.beta = form.beta;
  p.load_c = form.beta != 0.0;
  const int tiles = p.tiles_m * p.tiles_n;
  const int kblocks = plan.kblocks;
  p.kblocks = kblocks;
  p.c_prefetch = (dbg_flags & DGEMM_TEST_NO_C_PREFETCH) ? 0 : 1;
  p.split_k = plan.split_k;
  p.kblocks_per_split = plan.kblocks_per_split;
  p.dp_tiles = plan.dp_tiles;
  p.tail_tiles = plan.tail_tiles;
  p.tail_ipc = plan.tail_ipc;
  const int grid = plan.grid;
  p.tail_slot_base = 0;
  const bool uses_workspace = !cluster && (p.split_k > 1 || (p.tail_tiles > 0 && p.tail_ipc < kblocks));
  if (uses_workspace) {
    p.partial = static_cast<double*>(hold.workspace(kWorkspaceBytes));
    if (!p.partial) return DGEMM_ERR_CUDA;
  }

  CUtensorMap map_a, map_b;
  memset(&map_a, 0, sizeof(map_a));
  memset(&map_b, 0, sizeof(map_b));
  if (wants_tma) {
    if (form.native_at) {
      // A as stored, K x M: boxes of [16 k][16 rows of op(A)], one 3-D copy per stage when M is a multiple of 16
      p.a_blocked_map = (M % 16 == 0 && make_blocked_map(&map_a, A, K, M, lda, BK, bm / 16)) ? 1 : 0;
      if (!p.a_blocked_map && !make_map(&map_a, A, K, M, lda, 16, BK)) return DGEMM_ERR_CUDA;
    } else if (!make_map(&map_a, A, M, K, lda, BK, bm)) {
      return DGEMM_ERR_CUDA;
    }
    if (form.native_bt || form.native_at) {
      if (form.native_bt) {
        // B as stored, N x K: one box of 16 k x 128 rows (columns of op(B)) per stage, like an A tile
        if (!make_map(&map_b, B, N, K, ldb, BK, bn)) return DGEMM_ERR_CUDA;
      } else {
        p.b_blocked_map = (N % 16 == 0 && make_blocked_map(&map_b, B, K, N, ldb, BK, bn / 16)) ? 1 : 0;
        if (!p.b_blocked_map && !make_map(&map_b, B, K, N, ldb, 16, BK)) return DGEMM_ERR_CUDA;
      }
      const int which = cluster ? 3 : variant == DGEMM_VARIANT_TMA_WS ? (bm == 64 ? 1 : 0)
                        : bn == 64 ? 4 : bm == 256 ? 5 : bm == 32 ? 6 : 2;
      if (form.native_bt && form.native_at) launch_transposed_kernel<true, true>(which, grid, stream, map_a, map_b, p);
      else if (form.native_bt) launch_transposed_kernel<true, false>(which, grid, stream, map_a, map_b, p);
      else launch_transposed_kernel<false, true>(which, grid, stream, map_a, map_b, p);
    } else {
    p.b_blocked_map = (!(dbg_flags & DGEMM_TEST_NO_BLOCKED_B) && N % 16 == 0 && make_blocked_map(&map_b, B, K, N, ldb, BK, bn / 16)) ? 1 : 0;
    if (!p.b_blocked_map && !make_map(&map_b, B, K, N, ldb, 16, BK)) return DGEMM_ERR_CUDA;
    if (cluster)
      launch_cluster_pdl(dgemm_cluster_kernel<true, 64, 64, BN>, grid, p.split_k, TileCfg<64, 64, BN>::THREADS_,
                         (size_t)TileCfg<64, 64, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
    else if (variant == DGEMM_VARIANT_TMA_WS_BULK)
      launch_pdl(dgemm_dmma_wsb_kernel, dim3(grid), dim3(WsBulkCfg::THREADS_), (size_t)WsBulkCfg::SMEM_BYTES_, stream, map_a, map_b, p);
    else if (ws64)
      launch_gemm_kernel(dgemm_dmma_ws_kernel<true, 64>, grid, WsCfg<64>::THREADS_, WsCfg<64>::SMEM_BYTES_, stream, map_a, map_b, p);
    else if (variant == DGEMM_VARIANT_TMA_WS)
      launch_gemm_kernel(dgemm_dmma_ws_kernel<true>, grid, WS_THREADS, SMEM_BYTES, stream, map_a, map_b, p);
    else if (dfma)
      launch_dfma_kernel<true>(grid, stream, map_a, map_b, p);
    else
      launch_default_kernel<true>(bm, wtm, grid, stream, map_a, map_b, p);
    }
  } else {
    if (cluster)
      launch_cluster_pdl(dgemm_cluster_kernel<false, 64, 64, BN>, grid, p.split_k, TileCfg<64, 64, BN>::THREADS_,
                         (size_t)TileCfg<64, 64, BN>::SMEM_BYTES_, stream, map_a, map_b, p);
    else if (variant == DGEMM_VARIANT_GENERIC_WS)
      launch_gemm_kernel(dgemm_dmma_ws_kernel<false>, grid, WS_THREADS, SMEM_BYTES, stream, map_a, map_b, p);
    else if (dfma)
      launch_dfma_kernel<false>(grid, stream, map_a, map_b, p);
    else
      launch_default_kernel<false>(bm, wtm, grid, stream, map_a, map_b, p);
  }
  g_launches.fetch_add(1);
  if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  if (cluster) return DGEMM_OK;  // the K partitions were added inside the clusters
  if (p.split_k > 1) {
    launch_pdl(dgemm_splitk_reduce_kernel, dim3(tiles, REDUCE_CHUNKS), dim3(REDUCE_THREADS), 0, stream, p);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  }
  if (p.tail_tiles > 0 && p.tail_ipc < kblocks) {
    launch_pdl(dgemm_tail_reduce_kernel, dim3(p.tail_tiles, REDUCE_CHUNKS), dim3(REDUCE_THREADS), 0, stream, p);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  }
  return DGEMM_OK;
}

int launch_gemm(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                double* C, int64_t ldc, cudaStream_t stream, const GemmForm& form_in = GemmForm()) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  GemmForm form = form_in;

  int variant = g_variant.load();
  // The scratch this call needs (packed operands, partial tiles) is one lease of the device's pool,
  // held until the last kernel below has been enqueued: calls on other streams get other leases.
  scratch::Hold hold(st->scratch, stream);
  {
    // A transposed operand is always rewritten (row-major, 128-byte aligned rows) into the pack
    // buffer. An operand that TMA cannot address is repacked there when that is worth it: the copy
    // (16 bytes moved per packed element) small next to the arithmetic, the scratch moderate.
    const bool bad_a = !form.ta && (((uintptr_t)A & 15) != 0 || (lda % 2 != 0));
    const bool bad_b = !form.tb && (((uintptr_t)B & 15) != 0 || (ldb % 2 != 0));
    const int64_t plda = (K + 15) & ~(int64_t)15, pldb = (N + 15) & ~(int64_t)15;  // 128-byte aligned rows
    const size_t a_all = (size_t)M * plda * 8, b_all = (size_t)K * pldb * 8;
    bool pack_a = form.ta, pack_b = form.tb;
    if (variant == DGEMM_VARIANT_AUTO && (bad_a || bad_b) && !(g_test_flags.load() & DGEMM_TEST_NO_PACKING)) {
      const size_t bytes = ((pack_a || bad_a) ? a_all : 0) + ((pack_b || bad_b) ? b_all : 0);
      const double flop_per_byte = 2.0 * (double)M * (double)N * (double)K / (double)bytes;
      if (flop_per_byte >= (narrow_tiles_pay(M, N) ? kPackMinFlopPerByteNarrow : kPackMinFlopPerByte) && bytes <= kPackMaxBytes &&
          (2.0 * (double)M * (double)N * (double)K >= kPackMinFlop || (double)M * (double)N >= kPackMinElemsOfC)) {
        pack_a = pack_a || bad_a;
        pack_b = pack_b || bad_b;
      }
    }
    // A transposed operand that TMA can address as it is stored (16-byte aligned, even leading
    // dimension) needs no pass at all where the kernel that would run stages the transposed tile
    // itself: the library's own choice, no test flags, no forced split, the other operand addressable
    // (as it is, or after the packing pass decided above). Where the product is run as two products on a
    // column split of B (below), both parts' kernels have to be of that kind.
    if ((form.ta || form.tb) && st->bt_ok && variant == DGEMM_VARIANT_AUTO && g_test_flags.load() == 0 && g_split_k.load() <= 0 &&
        (!bad_a || pack_a) && (!bad_b || pack_b)) {
      const bool at_ok = form.ta && ((uintptr_t)A & 15) == 0 && (lda % 2 == 0);
      const bool bt_ok = form.tb && ((uintptr_t)B & 15) == 0 && (ldb % 2 == 0);
      // (the other transposed operand, if it cannot be used in place, is rewritten row-major and aligned)
      auto planned = [&](int64_t n) {
        return plan_gemm(M, n, K, true, variant, 0, 0, st->sm_count, st->two_ctas_ok, st->ws_ok, st->cluster_ok, false);
      };
      const int64_t r = N % BN;
      const bool supported = column_split_shape(M, N, K)
                                 ? plan_supports_native_bt(planned(N - r)) && plan_supports_native_bt(planned(r))
                                 : plan_supports_native_bt(planned(N));
      if (supported) {
        // B^T in the stage costs nothing measurable; A^T costs the arithmetic warps 0.5 % (four 8-byte loads
        // per fragment pair instead of two 16-byte ones), 1.2 % together with B^T, while the transposing
        // pass of A costs 0.7 % x 8192 / N: in place up to N = 8192, with B^T in place up to 4608
        if (bt_ok) { form.native_bt = true; pack_b = false; }
        if (at_ok && N <= (form.native_bt ? 4608 : 8192)) { form.native_at = true; pack_a = false; }
      }
    }
    if (pack_a || pack_b) {
      const size_t a_bytes = pack_a ? a_all : 0, b_bytes = pack_b ? b_all : 0;
      double* pa = static_cast<double*>(hold.pack_buffer(a_bytes + b_bytes + 256));
      if (!pa) return DGEMM_ERR_CUDA;
      double* pb = reinterpret_cast<double*>(reinterpret_cast<char*>(pa) + ((a_bytes + 255) & ~(size_t)255));
      if (pack_a && form.ta) {  // stored K x M
        dim3 grid((unsigned)((M + 31) / 32), grid_y((K + 31) / 32));
        launch_pdl(dgemm_transpose_kernel, grid, dim3(32, 8), 0, stream, A, (long long)lda, (int)K, (int)M, pa, (long long)plda);
        g_launches.fetch_add(1);
      }
      if (pack_b && form.tb) {  // stored N x K
        dim3 grid((unsigned)((K + 31) / 32), grid_y((N + 31) / 32));
        launch_pdl(dgemm_transpose_kernel, grid, dim3(32, 8), 0, stream, B, (long long)ldb, (int)N, (int)K, pb, (long long)pldb);
        g_launches.fetch_add(1);
      }
      // the plain copies of A and / or B: one launch
      PackOp ops[2];
      int nops = 0;
      int64_t gx = 0, gy = 0;
      if (pack_a && !form.ta) {
        ops[nops++] = PackOp{A, lda, (int)M, (int)K, pa, plda};
        gx = (K + 255) / 256;
        gy = (M + 7) / 8;
      }
      if (pack_b && !form.tb) {
        ops[nops++] = PackOp{B, ldb, (int)K, (int)N, pb, pldb};
        if ((N + 255) / 256 > gx) gx = (N + 255) / 256;
        if ((K + 7) / 8 > gy) gy = (K + 7) / 8;
      }
      if (nops > 0) {
        if (nops == 1) ops[1] = ops[0];
        launch_pdl(dgemm_pack2_kernel, dim3((unsigned)gx, grid_y(gy), (unsigned)nops), dim3(128), 0, stream, ops[0], ops[1]);
        g_launches.fetch_add(1);
      }
      if (pack_a) {
        A = pa;
        lda = plda;
      }
      if (pack_b) {
        B = pb;
        ldb = pldb;
      }
      if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
    }
  }
  // A column count just above a multiple of 128 on a large problem: the last tile column of 128
  // would be at most half full. The full tile columns and the remainder are run as two products on
  // disjoint columns of C, the remainder with the 256 x 32 tiles (2088^3: 573 -> 565 us, 4136^3: 4106
  // -> 4051 us; not worth it below: 1064^3 91 -> 100 us). The same for a tall problem with a few
  // tile columns, where the alternative is 128 x 64 tiles padded to the next 64 columns, when the
  // remainder fits one 32-column strip (6514 x 146 x 4096: 311 -> 271 us, 8192 x 129 x 8192: 764 ->
  // 642, 4000 x 400 x 4000: 433 -> 409; not below: 2600 x 140 x 2600 90 -> 94, 2000 x 140 x 2000 57 -> 66).
  // The sub-matrices start at a multiple of 128 columns, so whatever alignment B and C have is kept.
  if (variant == DGEMM_VARIANT_AUTO && g_test_flags.load() == 0 && g_split_k.load() <= 0) {
    const int64_t r = N % BN;
    const bool addressable = (((uintptr_t)A | (uintptr_t)B) & 15) == 0 && (lda % 2 == 0) && (ldb % 2 == 0);
    if (addressable && column_split_shape(M, N, K)) {
      rc = launch_gemm_packed(st, hold, variant, M, N - r, K, A, lda, B, ldb, C, ldc, stream, form);
      if (rc != DGEMM_OK) return rc;
      // (a B that is still the stored N x K matrix is cut by rows)
      const double* b_rest = form.native_bt ? B + (N - r) * ldb : B + (N - r);
      return launch_gemm_packed(st, hold, variant, M, r, K, A, lda, b_rest, ldb, C + (N - r), ldc, stream, form);
    }
  }
  return launch_gemm_packed(st, hold, variant, M, N, K, A, lda, B, ldb, C, ldc, stream, form);
}

// ---- split-K through a statically allocated workspace (no allocation at run time) --------------
//
// Some callers must not allocate device memory when they call into the library: code holding a
// lock that the allocator may also take, latency-critical loops with a fixed memory budget, or
// a process whose memory pool is owned by another component. For them the split-K partial tiles live in this file-scope device array.
// Every GPU that loads the library carries it (16 MiB) until the process exits.
constexpr int kStaticPartialTiles = 128;  // capacity: tiles * split_k partial tiles of 128 x 128 doubles
static __device__ __align__(256) double g_static_partials[(size_t)kStaticPartialTiles * BM * BN];

// Device address of g_static_partials per device. In host code the array's name is only a
// handle for the runtime, not an address a kernel could use; the address is looked up once per
// device, with that device current.
double* g_static_partials_addr[kMaxDevices];

int static_partials(double** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return DGEMM_ERR_DEVICE;
  }
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_static_partials_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_partials) != cudaSuccess || !ptr) {
      (void)cudaGetLastError();
      return DGEMM_ERR_CUDA;
    }
    g_static_partials_addr[dev] = static_cast<double*>(ptr);
  }
  *out = g_static_partials_addr[dev];
  return DGEMM_OK;
}

int launch_gemm_static_ws(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B,
                          int64_t ldb, double* C, int64_t ldc, int split_k, cudaStream_t stream) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);  // capability check, status word, shared-memory opt-in; allocates nothing
  if (rc != DGEMM_OK) return rc;
  double* partials = nullptr;
  rc = static_partials(&partials);
  if (rc != DGEMM_OK) return rc;

  const bool tma_ok = (((uintptr_t)A | (uintptr_t)B) & 15) == 0 && (lda % 2 == 0) && (ldb % 2 == 0);

  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  p.bm = BM;
  p.bn = BN;
  p.alpha = 1.0;
  p.beta = 1.0;
  p.load_c = 1;
  p.tiles_m = (int)((M + BM - 1) / BM);
  p.tiles_n = (int)((N + BN - 1) / BN);
  p.A = A; p.B = B; p.C = C;
  p.lda = lda; p.ldb = ldb; p.ldc = ldc;
  p.wait_limit_ns = kWaitLimitNs;
  p.status = st->status;
  p.group_m = 8;

  const int64_t tiles = (int64_t)p.tiles_m * p.tiles_n;
  const int kblocks = (int)((K + BK - 1) / BK);
  int64_t split = split_k;
  if (split <= 0) {
    // the library's choice: as many partitions as the SMs and the array can take, at least 4
    // k-blocks each; a problem too large for two partial tiles per output tile runs unsplit,
    // which needs no scratch at all
    split = st->sm_count / tiles;
    if (split > kblocks / 4) split = kblocks / 4;
    if (split > kStaticPartialTiles / tiles) split = kStaticPartialTiles / tiles;
    if (split < 2) split = (2 * tiles <= kStaticPartialTiles) ? 2 : 1;
  }
  if (split > kblocks) split = kblocks;
  p.kblocks = kblocks;
  p.dp_tiles = (int)tiles;  // uniform split-K over all tiles, no tail phase
  p.tail_tiles = 0;
  p.tail_ipc = 1;
  p.kblocks_per_split = (int)((kblocks + split - 1) / split);
  p.split_k = (kblocks + p.kblocks_per_split - 1) / p.kblocks_per_split;
  if (p.split_k > 1) {
    // the only use of the array; a call that ends up unsplit (split_k == 1, or a single k-block)
    // never touches it and has no size limit
    if (tiles * p.split_k > kStaticPartialTiles) return DGEMM_ERR_SIZE;
    p.partial = partials;  // every (tile, partition) slot in use is fully overwritten: nothing to clear
  }

  const int64_t units = tiles * p.split_k;
  const int grid = units < st->sm_count ? (int)units : st->sm_count;
  CUtensorMap map_a, map_b;
  memset(&map_a, 0, sizeof(map_a));
  memset(&map_b, 0, sizeof(map_b));
  if (tma_ok) {
    if (!make_map(&map_a, A, M, K, lda, BK, BM) || !make_map(&map_b, B, K, N, ldb, 16, BK)) return DGEMM_ERR_CUDA;
    launch_tile_kernel<true, 128, 64>(grid, stream, map_a, map_b, p);
  } else {
    launch_tile_kernel<false, 128, 64>(grid, stream, map_a, map_b, p);
  }
  g_launches.fetch_add(1);
  if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  if (p.split_k > 1) {
    dgemm_splitk_reduce_kernel<<<dim3((int)tiles, REDUCE_CHUNKS), REDUCE_THREADS, 0, stream>>>(p);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  }
  return DGEMM_OK;
}

// ---- FP64 issue-rate probe -------------------------------------------------------------------

__global__ void __launch_bounds__(256) fp64_probe_kernel(double* out, long long* cycles, int iters, double seed) {
  double c[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) { c[i][0] = i; c[i][1] = threadIdx.x; c[i][2] = 1.0; c[i][3] = 2.0; }
  const double a0 = seed, a1 = seed * 0.5, a2 = seed * 0.25, a3 = seed * 0.125, b0 = 1.0 - seed, b1 = 0.5 - seed;
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int i = 0; i < 8; ++i) ptx::dmma_m16n8k8(c[i], a0, a1, a2, a3, b0, b1);
  }
  const long long t1 = clock64();
  double r = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) r += c[i][0] + c[i][1] + c[i][2] + c[i][3];
  out[blockIdx.x * blockDim.x + threadIdx.x] = r;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

// The same for plain FP64 fused multiply-adds: 16 independent chains per thread, 512 threads per SM.
__global__ void __launch_bounds__(512) fp64_fma_probe_kernel(double* out, long long* cycles, int iters, double seed) {
  double c[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) c[i] = i + threadIdx.x;
  const double a = seed, b = 1.0 - seed;
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int i = 0; i < 16; ++i) c[i] = fma(c[i], a, b);
  }
  const long long t1 = clock64();
  double r = 0.0;
#pragma unroll
  for (int i = 0; i < 16; ++i) r += c[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = r;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

int run_fp64_probe(bool plain_fma, int millis, double* fma_per_clk_sm, double* tflops) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  if (millis < 1) millis = 1;
  if (millis > 10000) millis = 10000;
  const int blocks = st->sm_count, threads = plain_fma ? 512 : 256;
  double* out = nullptr;
  long long* cyc = nullptr;
  auto launch = [&](int iters) {
    if (plain_fma) fp64_fma_probe_kernel<<<blocks, threads>>>(out, cyc, iters, 0.999999);
    else fp64_probe_kernel<<<blocks, threads>>>(out, cyc, iters, 0.999999);
  };
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  rc = DGEMM_ERR_CUDA;
  do {
    if (cudaMalloc(reinterpret_cast<void**>(&out), sizeof(double) * blocks * threads) != cudaSuccess) break;
    if (cudaMalloc(reinterpret_cast<void**>(&cyc), sizeof(long long) * blocks) != cudaSuccess) break;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) break;
    // calibrate with a short run, then size the timed run to about `millis`
    int iters = 2000;
    float ms = 0.f;
    launch(iters);
    if (cudaEventRecord(e0) != cudaSuccess) break;
    launch(iters);
    if (cudaEventRecord(e1) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) break;
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) break;
    double scale = millis / ms;
    if (scale > 100000.0) scale = 100000.0;
    iters = (int)(iters * scale) + 1;
    if (cudaEventRecord(e0) != cudaSuccess) break;
    launch(iters);
    if (cudaEventRecord(e1) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess) break;
    if (cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess) break;
    g_launches.fetch_add(3);
    long long* h = static_cast<long long*>(malloc(sizeof(long long) * blocks));
    if (!h) break;
    if (cudaMemcpy(h, cyc, sizeof(long long) * blocks, cudaMemcpyDeviceToHost) != cudaSuccess) { free(h); break; }
    long long mx = 1;
    for (int i = 0; i < blocks; ++i) if (h[i] > mx) mx = h[i];
    free(h);
    // per warp and iteration: 8 MMAs of 16*8*8 = 1024 fused multiply-adds, or 64 FMA instructions of 32 lanes
    const double fma_per_block = (double)(threads / 32) * iters * (plain_fma ? 64.0 * 32.0 : 8.0 * 1024.0);
    if (fma_per_clk_sm) *fma_per_clk_sm = fma_per_block / (double)mx;
    if (tflops) *tflops = 2.0 * fma_per_block * blocks / (ms * 1e-3) / 1e12;
    rc = DGEMM_OK;
  } while (0);
  if (rc != DGEMM_OK) (void)cudaGetLastError();
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (out) cudaFree(out);
  if (cyc) cudaFree(cyc);
  return rc;
}

}  // namespace

extern "C" {

int dgemm_f64(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb, double* C,
              int64_t ldc, void* stream) {
  const int v = validate(M, N, K, A, lda, B, ldb, C, ldc);
  if (v == 1) return DGEMM_OK;
  if (v != DGEMM_OK) return v;
  return launch_gemm(M, N, K, A, lda, B, ldb, C, ldc, static_cast<cudaStream_t>(stream));
}

int dgemm_f64_ex(int transa, int transb, int64_t M, int64_t N, int64_t K, double alpha, const double* A, int64_t lda,
                 const double* B, int64_t ldb, double beta, double* C, int64_t ldc, void* stream) {
  if ((transa != DGEMM_OP_N && transa != DGEMM_OP_T) || (transb != DGEMM_OP_N && transb != DGEMM_OP_T))
    return DGEMM_ERR_BAD_DIM;
  GemmForm form;
  form.ta = transa == DGEMM_OP_T;
  form.tb = transb == DGEMM_OP_T;
  form.alpha = alpha;
  form.beta = beta;
  const int v = validate(M, N, K, A, lda, B, ldb, C, ldc, form.ta, form.tb, beta != 1.0, alpha == 0.0);
  if (v == 1) return DGEMM_OK;
  if (v < 0) return v;
  if (v == 2) {  // no product: C = beta * C
    DeviceState* st = nullptr;
    const int rc = device_state(&st);
    if (rc != DGEMM_OK) return rc;
    const unsigned rows = (unsigned)(M < 4096 ? M : 4096);
    dgemm_scale_kernel<<<dim3((unsigned)((N + 255) / 256), rows), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        C, ldc, (int)M, (int)N, beta);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? DGEMM_OK : DGEMM_ERR_CUDA;
  }
  return launch_gemm(M, N, K, A, lda, B, ldb, C, ldc, static_cast<cudaStream_t>(stream), form);
}

int dgemm_f64_static_ws(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                        double* C, int64_t ldc, int split_k, void* stream) {
  if (split_k < 0) return DGEMM_ERR_VARIANT;
  const int v = validate(M, N, K, A, lda, B, ldb, C, ldc);
  if (v == 1) return DGEMM_OK;
  if (v != DGEMM_OK) return v;
  return launch_gemm_static_ws(M, N, K, A, lda, B, ldb, C, ldc, split_k, static_cast<cudaStream_t>(stream));
}

int dgemm_f64_host(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                   double* C, int64_t ldc) {
  const int v = validate(M, N, K, A, lda, B, ldb, C, ldc);
  if (v == 1) return DGEMM_OK;
  if (v != DGEMM_OK) return v;
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;

  // Dense device copies with even leading dimensions (keeps the TMA path available). A and C
  // travel in blocks of rows through a few buffers, on three streams, so that the upload of later
  // blocks, the arithmetic of block i and the download of block i-1 overlap.
  cudaMemPool_t pool = nullptr;
  rc = ensure_host_pool(st, &pool);
  if (rc != DGEMM_OK) return rc;
  const int64_t dlda = K + (K & 1), dldb = N + (N & 1), dldc = N + (N & 1);
  const int64_t blk = (M > 2 * kHostBlockRows) ? kHostBlockRows : M;  // rows per block
  const int64_t nblk = (M + blk - 1) / blk;
  // B travels in panels of kHostPanelRows rows (whole rows: contiguous in host memory when
  // ldb == N) behind the first `heads` blocks of A and C, and those blocks are multiplied K panel
  // by K panel as the panels arrive, each product added into its block of C: the arithmetic
  // starts after 0.5 GB instead of 0.7 GB (8192^3) have crossed the host link, and by the time B
  // is complete three eighths of it are done. The other blocks follow through a ring of buffers.
  // The head blocks' C does not wait in front of all that: their first panel product is written
  // with beta = 0, the caller's C follows B across the link into buffers of its own and is added
  // to the finished product (one rounding, as in the kernels' own epilogue).
  const int64_t prows = (nblk > 1 && K > 2 * kHostPanelRows) ? kHostPanelRows : K;
  const int64_t npan = (K + prows - 1) / prows;
  const int heads = (npan > 1 && nblk >= 6) ? 3 : 1;
  const int nbuf = nblk > 1 ? (int)((nblk < heads + 2) ? nblk : heads + 2) : 1;
  cudaStream_t s_up = nullptr, s_run = nullptr, s_down = nullptr;
  double* dB = nullptr;
  double* dA[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  double* dC[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  double* dT[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr};  // the caller's C of the head blocks
  std::vector<cudaEvent_t> ev_pan;  // one per row panel of B
  cudaEvent_t ev_alloc = nullptr, ev_up[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr},
              ev_run[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr},
              ev_down[kHostMaxBufs] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  rc = DGEMM_ERR_CUDA;
  do {
    if (cudaStreamCreateWithFlags(&s_up, cudaStreamNonBlocking) != cudaSuccess) break;
    if (cudaStreamCreateWithFlags(&s_run, cudaStreamNonBlocking) != cudaSuccess) break;
    if (cudaStreamCreateWithFlags(&s_down, cudaStreamNonBlocking) != cudaSuccess) break;
    bool ok = cudaEventCreateWithFlags(&ev_alloc, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < nbuf && ok; ++i)
      ok = cudaEventCreateWithFlags(&ev_up[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev_run[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev_down[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) break;
    if (cudaMallocFromPoolAsync(reinterpret_cast<void**>(&dB), (size_t)K * dldb * 8, pool, s_up) != cudaSuccess) break;
    for (int i = 0; i < nbuf && ok; ++i)
      ok = cudaMallocFromPoolAsync(reinterpret_cast<void**>(&dA[i]), (size_t)blk * dlda * 8, pool, s_up) == cudaSuccess &&
           cudaMallocFromPoolAsync(reinterpret_cast<void**>(&dC[i]), (size_t)blk * dldc * 8, pool, s_up) == cudaSuccess;
    const bool late_c = npan > 1;  // (heads > 1 implies it)
    for (int h = 0; h < heads && ok && late_c; ++h)
      ok = cudaMallocFromPoolAsync(reinterpret_cast<void**>(&dT[h]), (size_t)blk * dldc * 8, pool, s_up) == cudaSuccess;
    if (!ok) break;
    // the other streams may touch the buffers only after the (stream-ordered) allocations
    if (cudaEventRecord(ev_alloc, s_up) != cudaSuccess) break;
    if (cudaStreamWaitEvent(s_run, ev_alloc, 0) != cudaSuccess || cudaStreamWaitEvent(s_down, ev_alloc, 0) != cudaSuccess) break;
    int inner = DGEMM_OK;
    auto upload_block = [&](int64_t i, bool with_c) -> bool {
      const int b = (int)(i % nbuf);
      const int64_t r0 = i * blk, rows = (M - r0 < blk) ? M - r0 : blk;
      // buffer b is free again once block i - 2 has been downloaded
      if (i >= nbuf && cudaStreamWaitEvent(s_up, ev_down[b], 0) != cudaSuccess) return false;
      return cudaMemcpy2DAsync(dA[b], dlda * 8, A + r0 * lda, lda * 8, K * 8, rows, cudaMemcpyHostToDevice, s_up) == cudaSuccess &&
             (!with_c ||
              cudaMemcpy2DAsync(dC[b], dldc * 8, C + r0 * ldc, ldc * 8, N * 8, rows, cudaMemcpyHostToDevice, s_up) == cudaSuccess) &&
             cudaEventRecord(ev_up[b], s_up) == cudaSuccess;
    };
    bool heads_up = true;
    for (int h = 0; h < heads && heads_up; ++h)
      heads_up = upload_block(h, !late_c) && cudaStreamWaitEvent(s_run, ev_up[h], 0) == cudaSuccess;
    if (!heads_up) break;
    ev_pan.assign((size_t)npan, nullptr);
    for (int64_t j = 0; j < npan && inner == DGEMM_OK; ++j) {
      const int64_t k0 = j * prows, krows = (K - k0 < prows) ? K - k0 : prows;
      if (cudaEventCreateWithFlags(&ev_pan[(size_t)j], cudaEventDisableTiming) != cudaSuccess ||
          cudaMemcpy2DAsync(dB + k0 * dldb, dldb * 8, B + k0 * ldb, ldb * 8, N * 8, krows, cudaMemcpyHostToDevice, s_up) != cudaSuccess ||
          cudaEventRecord(ev_pan[(size_t)j], s_up) != cudaSuccess || cudaStreamWaitEvent(s_run, ev_pan[(size_t)j], 0) != cudaSuccess) {
        inner = DGEMM_ERR_CUDA;
        break;
      }
      GemmForm form;  // the first panel product overwrites the buffer, the others add to it
      form.beta = (j == 0) ? 0.0 : 1.0;
      for (int h = 0; h < heads && npan > 1 && inner == DGEMM_OK; ++h)
        inner = launch_gemm(blk < M ? blk : M, N, krows, dA[h] + k0, dlda, dB + k0 * dldb, dldb, dC[h], dldc, s_run, form);
    }
    if (inner != DGEMM_OK) { rc = inner; break; }
    // Behind B the link carries, in this order: block `heads`, the caller's C of head block 0, block
    // `heads + 1`, the C of the other head blocks, then the remaining blocks. The arithmetic goes
    // straight from the last panel product into block `heads` (whose rows are there by then), and
    // head block 0 is finished and downloaded early enough to free its buffers for the ring.
    // (The events ev_up[h] of the head blocks are free again: s_run has consumed them.)
    int64_t uploaded = heads;  // blocks [0, uploaded) have been sent
    auto upload_head_c = [&](int h) -> bool {
      const int64_t r0 = (int64_t)h * blk, rows = (M - r0 < blk) ? M - r0 : blk;
      return cudaMemcpy2DAsync(dT[h], dldc * 8, C + r0 * ldc, ldc * 8, N * 8, rows, cudaMemcpyHostToDevice, s_up) == cudaSuccess &&
             cudaEventRecord(ev_up[h], s_up) == cudaSuccess;
    };
    if (late_c) {
      bool sent = true;
      if (cudaEventRecord(ev_alloc, s_run) != cudaSuccess) sent = false;  // (reused: behind the last panel product)
      if (sent && uploaded < nblk && uploaded < nbuf) sent = upload_block(uploaded++, true);
      if (sent) sent = upload_head_c(0);
      if (sent && uploaded < nblk && uploaded < nbuf) sent = upload_block(uploaded++, true);
      for (int h = 1; h < heads && sent; ++h) sent = upload_head_c(h);
      if (!sent) { rc = DGEMM_ERR_CUDA; break; }
    }
    for (int64_t i = 0; i < nblk; ++i) {
      const int b = (int)(i % nbuf);
      const int64_t r0 = i * blk, rows = (M - r0 < blk) ? M - r0 : blk;
      if (i < heads && late_c) {
        // a head block: its product is complete; add the caller's C and send it back, all on the
        // download stream, so that the arithmetic stream never waits for that C
        if (cudaStreamWaitEvent(s_down, ev_alloc, 0) != cudaSuccess || cudaStreamWaitEvent(s_down, ev_up[b], 0) != cudaSuccess) {
          inner = DGEMM_ERR_CUDA;
          break;
        }
        const unsigned gy = (unsigned)(rows < 4096 ? rows : 4096);
        dgemm_add_kernel<<<dim3((unsigned)((dldc / 2 + 255) / 256), gy), 256, 0, s_down>>>(dC[b], dldc, dT[b], dldc, (int)rows, (int)dldc);
        g_launches.fetch_add(1);
        if (cudaGetLastError() != cudaSuccess ||
            cudaMemcpy2DAsync(C + r0 * ldc, ldc * 8, dC[b], dldc * 8, N * 8, rows, cudaMemcpyDeviceToHost, s_down) != cudaSuccess ||
            cudaEventRecord(ev_down[b], s_down) != cudaSuccess) {
          inner = DGEMM_ERR_CUDA;
          break;
        }
        continue;
      }
      if (i >= uploaded) {
        if (!upload_block(i, true)) { inner = DGEMM_ERR_CUDA; break; }
        uploaded = i + 1;
      }
      if (i >= heads && cudaStreamWaitEvent(s_run, ev_up[b], 0) != cudaSuccess) { inner = DGEMM_ERR_CUDA; break; }
      // The last block of a long run is multiplied and sent back in two halves: nothing overlaps
      // with the very last download, so it should be short (8192^3: 0.5 ms of 38).
      const bool halves = i == nblk - 1 && i >= heads && nblk >= 6 && rows >= 512;
      const int64_t part[3] = {0, halves ? rows / 2 : rows, rows};
      for (int q = 0; q < (halves ? 2 : 1) && inner == DGEMM_OK; ++q) {
        const int64_t q0 = part[q], qrows = part[q + 1] - part[q];
        if (i >= heads || npan == 1)
          inner = launch_gemm(qrows, N, K, dA[b] + q0 * dlda, dlda, dB, dldb, dC[b] + q0 * dldc, dldc, s_run);
        if (inner != DGEMM_OK) break;
        if (cudaEventRecord(ev_run[b], s_run) != cudaSuccess || cudaStreamWaitEvent(s_down, ev_run[b], 0) != cudaSuccess ||
            cudaMemcpy2DAsync(C + (r0 + q0) * ldc, ldc * 8, dC[b] + q0 * dldc, dldc * 8, N * 8, qrows, cudaMemcpyDeviceToHost, s_down) != cudaSuccess ||
            cudaEventRecord(ev_down[b], s_down) != cudaSuccess)
          inner = DGEMM_ERR_CUDA;
      }
      if (inner != DGEMM_OK) break;
    }
    if (inner != DGEMM_OK) { rc = inner; break; }
    if (cudaStreamSynchronize(s_down) != cudaSuccess || cudaStreamSynchronize(s_run) != cudaSuccess ||
        cudaStreamSynchronize(s_up) != cudaSuccess)
      break;
    rc = DGEMM_OK;
  } while (0);
  if (rc != DGEMM_OK) (void)cudaGetLastError();
  // everything that used the buffers has finished (or failed) before they go back to the pool
  if (s_run) cudaStreamSynchronize(s_run);
  if (s_down) cudaStreamSynchronize(s_down);
  if (s_up) {
    if (dB) cudaFreeAsync(dB, s_up);
    for (int i = 0; i < kHostMaxBufs; ++i) {
      if (dA[i]) cudaFreeAsync(dA[i], s_up);
      if (dC[i]) cudaFreeAsync(dC[i], s_up);
      if (dT[i]) cudaFreeAsync(dT[i], s_up);
    }
    cudaStreamSynchronize(s_up);
  }
  if (ev_alloc) cudaEventDestroy(ev_alloc);
  for (cudaEvent_t e : ev_pan)
    if (e) cudaEventDestroy(e);
  for (int i = 0; i < kHostMaxBufs; ++i) {
    if (ev_up[i]) cudaEventDestroy(ev_up[i]);
    if (ev_run[i]) cudaEventDestroy(ev_run[i]);
    if (ev_down[i]) cudaEventDestroy(ev_down[i]);
  }
  if (s_up) cudaStreamDestroy(s_up);
  if (s_run) cudaStreamDestroy(s_run);
  if (s_down) cudaStreamDestroy(s_down);
  return rc;
}

const char* dgemm_strerror(int status) {
  switch (status) {
    case DGEMM_OK: return "success";
    case DGEMM_ERR_BAD_DIM: return "M, N or K is negative or too large";
    case DGEMM_ERR_BAD_LD: return "a leading dimension is smaller than the row length";
    case DGEMM_ERR_NULL: return "a required pointer is NULL";
    case DGEMM_ERR_ALIGN: return "a pointer is not 8-byte aligned";
    case DGEMM_ERR_ALIAS: return "C overlaps A or B";
    case DGEMM_ERR_DEVICE: return "no CUDA device, or the current device is not compute capability 10.x";
    case DGEMM_ERR_CUDA: return "a CUDA runtime or driver call failed";
    case DGEMM_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case DGEMM_ERR_VARIANT: return "unknown kernel variant, or the forced variant cannot run these operands";
    case DGEMM_ERR_SIZE: return "problem exceeds the fixed capacity of this entry point";
    default: return "unknown status";
  }
}

int dgemm_version(void) { return 100; /* 0.1.0 */ }

int dgemm_plan(int64_t M, int64_t N, int64_t K, int tma_addressable, int sm_count, int* out) {
  if (!out) return DGEMM_ERR_NULL;
  if (M <= 0 || N <= 0 || K <= 0 || M > INT32_MAX - 512 || N > INT32_MAX - 512 || K > INT32_MAX - 512) return DGEMM_ERR_BAD_DIM;
  const bool ws_ok[4] = {true, true, true, true};
  const Plan pl = plan_gemm(M, N, K, tma_addressable != 0, g_variant.load(), g_test_flags.load(), g_split_k.load(),
                            sm_count > 0 ? sm_count : 148, true, ws_ok, true, tma_addressable != 0);
  if (pl.status != DGEMM_OK) return pl.status;
  const int v[12] = {pl.variant, pl.bm, pl.bn, pl.wtm, pl.ctas_per_sm, pl.grid, pl.kblocks, pl.split_k,
                     pl.kblocks_per_split, pl.dp_tiles, pl.tail_tiles, pl.tail_ipc};
  for (int i = 0; i < 12; ++i) out[i] = v[i];
  return DGEMM_OK;
}

int dgemm_set_variant(int variant) {
  if (variant < DGEMM_VARIANT_AUTO || variant >= DGEMM_VARIANT_COUNT) return DGEMM_ERR_VARIANT;
  g_variant.store(variant);
  return DGEMM_OK;
}

int dgemm_set_test_flags(int flags) {
  constexpr int kAll = DGEMM_TEST_NO_C_PREFETCH | DGEMM_TEST_NO_BLOCKED_B | DGEMM_TEST_TALL_TILES | DGEMM_TEST_SMALL_WARP_TILES |
                       DGEMM_TEST_NO_PACKING | DGEMM_TEST_WS_TWO_CTAS | DGEMM_TEST_NO_CLUSTER | DGEMM_TEST_DROP_LOADS;
  if (flags < 0 || (flags & ~kAll) != 0) return DGEMM_ERR_VARIANT;
  g_test_flags.store(flags);
  return DGEMM_OK;
}

int dgemm_set_test_wait_limit(int limit_us) {
  if (limit_us < 0 || limit_us > 4000000) return DGEMM_ERR_VARIANT;
  g_test_wait_limit_ns.store((long long)limit_us * 1000ll);
  return DGEMM_OK;
}

int dgemm_set_split_k(int split_k) {
  if (split_k < 0) return DGEMM_ERR_VARIANT;
  g_split_k.store(split_k);
  return DGEMM_OK;
}

int dgemm_last_device_status(void* stream) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    (void)cudaGetLastError();
    return DGEMM_ERR_CUDA;
  }
  int word = 0;
  if (cudaMemcpy(&word, st->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return DGEMM_ERR_CUDA;
  if (word != 0 && cudaMemset(st->status, 0, sizeof(int)) != cudaSuccess) return DGEMM_ERR_CUDA;
  return word;
}

int dgemm_release_scratch(void) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  if (cudaDeviceSynchronize() != cudaSuccess) {
    (void)cudaGetLastError();
    return DGEMM_ERR_CUDA;
  }
  bool ok = scratch::release_all(st->scratch);
  std::lock_guard<std::mutex> lock(g_mutex);
  if (st->host_pool) ok = cudaMemPoolTrimTo(st->host_pool, 0) == cudaSuccess && ok;
  if (!ok) (void)cudaGetLastError();
  return ok ? DGEMM_OK : DGEMM_ERR_CUDA;
}

int64_t dgemm_launch_count(void) { return g_launches.load(); }

int dgemm_selftest_wait_timeout(int limit_us) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  if (limit_us < 1) limit_us = 1;
  if (limit_us > 1000000) limit_us = 1000000;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.wait_limit_ns = (unsigned long long)limit_us * 1000ull;
  p.status = st->status;
  int* gave_up = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&gave_up), sizeof(int)) != cudaSuccess) return DGEMM_ERR_CUDA;
  int host_gave_up = 0;
  rc = DGEMM_ERR_CUDA;
  do {
    if (cudaMemset(gave_up, 0, sizeof(int)) != cudaSuccess) break;
    dgemm_wait_timeout_selftest_kernel<<<1, 64>>>(p, gave_up);
    g_launches.fetch_add(1);
    if (cudaGetLastError() != cudaSuccess) break;
    if (cudaDeviceSynchronize() != cudaSuccess) break;
    if (cudaMemcpy(&host_gave_up, gave_up, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) break;
    rc = DGEMM_OK;
  } while (0);
  cudaFree(gave_up);
  if (rc != DGEMM_OK) return rc;
  // all 64 threads must have left their wait; the status word (read by dgemm_last_device_status) says why
  return host_gave_up == 64 ? DGEMM_OK : DGEMM_ERR_CUDA;
}

int dgemm_fp64_peak_probe(int millis, double* fma_per_clk_sm, double* tflops) {
  return run_fp64_probe(false, millis, fma_per_clk_sm, tflops);
}

int dgemm_fp64_fma_probe(int millis, double* fma_per_clk_sm, double* tflops) {
  return run_fp64_probe(true, millis, fma_per_clk_sm, tflops);
}

}  // extern "C"
