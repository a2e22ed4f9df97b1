// C ABI of the single-precision entry point (include/sgemm.h): validation, packing of operands
// TMA cannot address, tensor maps, launch of sgemm_ffma_kernel.
#include <cstdint>
#include <cstring>
#include <mutex>
#include <utility>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/sgemm.h"
#include "scratch_pool.h"
#include "sgemm_ffma.cuh"

namespace {

using namespace sgemm;

constexpr int kMaxDevices = 64;
constexpr unsigned long long kWaitLimitNs = 4000000000ull;  // bounded device-side waits give up after 4 s

__device__ int g_sgemm_status_word;

struct DeviceState {
  bool ready = false;
  int sm_count = 0;
  int* status = nullptr;
  scratch::Pool scratch;  // stream-K partial tiles and packed operand copies, leased per call (scratch_pool.h)
};

DeviceState g_dev[kMaxDevices];
std::mutex g_mutex;

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

template <int RPT, int NH>
bool configure_kernel() {
  return cudaFuncSetAttribute(sgemm_ffma_kernel<RPT, NH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              Cfg<RPT, NH>::SMEM_BYTES) == cudaSuccess;
}

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
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&st.status), g_sgemm_status_word) != cudaSuccess) return DGEMM_ERR_CUDA;
    if (cudaMemset(st.status, 0, sizeof(int)) != cudaSuccess) return DGEMM_ERR_CUDA;
    if (!configure_kernel<16, 2>() || !configure_kernel<8, 2>() || !configure_kernel<4, 2>() ||
        !configure_kernel<16, 1>() || !configure_kernel<8, 1>() || !configure_kernel<4, 1>())
      return DGEMM_ERR_CUDA;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
          qres != cudaDriverEntryPointSuccess)
        return DGEMM_ERR_CUDA;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    st.sm_count = sms;
    st.ready = true;
  }
  *out = &st;
  return DGEMM_OK;
}

// 2-D f32 tensor map: inner extent `cols`, outer extent `rows` with stride ld floats; 128-byte
// swizzle; elements outside the matrix read as zero.
bool make_map(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, int64_t ld, int box_cols, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * sizeof(float)};
  const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D view of a row-major K x N matrix whose N is a multiple of 32: (column within a block of 32,
// k, block of 32 columns). One copy of box 32 x TK x (tile columns / 32) lands as consecutive
// [TK][32] sub-tiles.
bool make_blocked_map(CUtensorMap* map, const float* base, int64_t K, int64_t N, int64_t ld, int tile_cols) {
  const cuuint64_t dims[3] = {32, (cuuint64_t)K, (cuuint64_t)(N / 32)};
  const cuuint64_t strides[2] = {(cuuint64_t)ld * sizeof(float), 32 * sizeof(float)};
  const cuuint32_t box[3] = {32, (cuuint32_t)TK, (cuuint32_t)(tile_cols / 32)};
  const cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool ranges_overlap(const void* p, int64_t pbytes, const void* q, int64_t qbytes) {
  const uintptr_t a = (uintptr_t)p, b = (uintptr_t)q;
  return a < b + (uintptr_t)qbytes && b < a + (uintptr_t)pbytes;
}

// Everything that can be decided without touching the device. Returns 1 for "nothing to do".
int validate(int64_t M, int64_t N, int64_t K, const float* A, int64_t lda, const float* B, int64_t ldb, const float* C,
             int64_t ldc) {
  const int64_t kMaxDim = (int64_t)INT32_MAX - 2 * MAX_TM;
  if (M < 0 || N < 0 || K < 0 || M > kMaxDim || N > kMaxDim || K > kMaxDim) return DGEMM_ERR_BAD_DIM;
  if (M == 0 || N == 0) return 1;
  if (lda < (K > 0 ? K : 1) || ldb < N || ldc < N) return DGEMM_ERR_BAD_LD;
  if (K == 0) return 1;
  if (!A || !B || !C) return DGEMM_ERR_NULL;
  if (((uintptr_t)A | (uintptr_t)B | (uintptr_t)C) & 3) return DGEMM_ERR_ALIGN;
  const int64_t abytes = ((M - 1) * lda + K) * 4, bbytes = ((K - 1) * ldb + N) * 4, cbytes = ((M - 1) * ldc + N) * 4;
  if (ranges_overlap(C, cbytes, A, abytes) || ranges_overlap(C, cbytes, B, bbytes)) return DGEMM_ERR_ALIAS;
  const int64_t tiles = ((M + 63) / 64) * ((N + 63) / 64);  // (the smallest tile)
  if (tiles > (int64_t)INT32_MAX / 2) return DGEMM_ERR_BAD_DIM;
  return DGEMM_OK;
}

// Launch with programmatic stream serialization (the kernels wait with griddepcontrol.wait before
// their first global access): hides a few microseconds of launch latency per kernel.
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

template <int RPT, int NH>
void launch_kernel(int grid, cudaStream_t stream, const CUtensorMap& map_a, const CUtensorMap& map_b, const Params& p) {
  launch_pdl(sgemm_ffma_kernel<RPT, NH>, dim3(grid), dim3(THREADS), (size_t)Cfg<RPT, NH>::SMEM_BYTES, stream, map_a, map_b, p);
}

inline unsigned grid_y(int64_t blocks) { return (unsigned)(blocks < 65535 ? blocks : 65535); }

int launch(int64_t M, int64_t N, int64_t K, const float* A, int64_t lda, const float* B, int64_t ldb, float* C, int64_t ldc,
           cudaStream_t stream) {
  DeviceState* st = nullptr;
  int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;

  // scratch of this call: one lease of the device's pool, held until the last launch below
  scratch::Hold hold(st->scratch, stream);
  // operands TMA cannot address are repacked (16-byte aligned base, rows of a multiple of 128 bytes)
  const bool pack_a = ((uintptr_t)A & 15) != 0 || (lda % 4 != 0);
  const bool pack_b = ((uintptr_t)B & 15) != 0 || (ldb % 4 != 0);
  if (pack_a || pack_b) {
    const int64_t plda = (K + 31) & ~(int64_t)31, pldb = (N + 31) & ~(int64_t)31;
    const size_t a_bytes = pack_a ? (size_t)M * plda * 4 : 0, b_bytes = pack_b ? (size_t)K * pldb * 4 : 0;
    float* pa = static_cast<float*>(hold.pack_buffer(a_bytes + b_bytes + 256));
    if (!pa) return DGEMM_ERR_CUDA;
    float* pb = reinterpret_cast<float*>(reinterpret_cast<char*>(pa) + ((a_bytes + 255) & ~(size_t)255));
    PackOpF ops[2];
    int nops = 0;
    int64_t gx = 0, gy = 0;
    if (pack_a) {
      ops[nops++] = PackOpF{A, lda, (int)M, (int)K, pa, plda};
      gx = (K + 255) / 256;
      gy = M;
      A = pa;
      lda = plda;
    }
    if (pack_b) {
      ops[nops++] = PackOpF{B, ldb, (int)K, (int)N, pb, pldb};
      if ((N + 255) / 256 > gx) gx = (N + 255) / 256;
      if (K > gy) gy = K;
      B = pb;
      ldb = pldb;
    }
    if (nops == 1) ops[1] = ops[0];
    launch_pdl(sgemm_pack_kernel, dim3((unsigned)gx, grid_y(gy), (unsigned)nops), dim3(256), 0, stream, ops[0], ops[1]);
    if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  }

  Params p;
  memset(&p, 0, sizeof(p));
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  // 128-row tiles when 256-row tiles would compute at least a tenth more rows
  const int64_t pad128 = (M + 127) / 128 * 128, pad256 = (M + 255) / 256 * 256;
  // ... and 64-row tiles for a short M (at most 64 rows, or 129..192) that they fit better still
  const int64_t pad64 = (M + 63) / 64 * 64;
  const int TM = (M <= 192 && pad64 < pad128) ? 64 : ((double)pad128 * 1.10 <= (double)pad256) ? 128 : 256;
  // 64-column tiles for a narrow N that they fit better (at most 64 columns, or 129..192)
  const int TNV = (N <= 192 && (N + 63) / 64 * 64 < (N + 127) / 128 * 128) ? 64 : 128;
  p.tm_rows = TM;
  p.tn_cols = TNV;
  p.tiles_m = (int)((M + TM - 1) / TM);
  p.tiles_n = (int)((N + TNV - 1) / TNV);
  p.kblocks = (int)((K + TK - 1) / TK);
  p.group_m = 8;  // 1024 rows per raster group
  p.A = A; p.B = B; p.C = C;
  p.lda = lda; p.ldb = ldb; p.ldc = ldc;
  p.wait_limit_ns = kWaitLimitNs;
  p.status = st->status;

  CUtensorMap map_a, map_b;
  memset(&map_a, 0, sizeof(map_a));
  memset(&map_b, 0, sizeof(map_b));
  if (!make_map(&map_a, A, M, K, lda, TK, TM)) return DGEMM_ERR_CUDA;
  p.b_blocked_map = (N % 32 == 0 && make_blocked_map(&map_b, B, K, N, ldb, TNV)) ? 1 : 0;
  if (!p.b_blocked_map && !make_map(&map_b, B, K, N, ldb, 32, TK)) return DGEMM_ERR_CUDA;

  // whole waves of tiles run data-parallel; the last partial wave is spread evenly over the CTAs
  // (stream-K) when that saves more time than the partial-tile round trip costs
  const int tiles = p.tiles_m * p.tiles_n;
  const int resident = st->sm_count;
  int grid = tiles < resident ? tiles : resident;
  p.dp_tiles = tiles;
  p.tail_tiles = 0;
  p.tail_ipc = p.kblocks;
  const int tail = tiles % resident;
  if (tail > 0 && p.kblocks >= 2 && (1.0 - (double)tail / resident) * p.kblocks >= 3.0 &&
      (long long)(tail + 1) * p.kblocks < (long long)INT32_MAX) {
    p.dp_tiles = tiles - tail;
    p.tail_tiles = tail;
    const long long total = (long long)tail * p.kblocks;
    long long ipc = (total + resident - 1) / resident;
    if (ipc > p.kblocks) ipc = p.kblocks;
    p.tail_ipc = (int)ipc;
    const int span_ctas = (int)((total + ipc - 1) / ipc);
    if (p.dp_tiles == 0) grid = span_ctas < resident ? span_ctas : resident;
    p.partial = static_cast<float*>(hold.workspace((size_t)2 * resident * MAX_TM * TN * sizeof(float)));
    if (!p.partial) return DGEMM_ERR_CUDA;
  }
  if (TNV == 128) {
    if (TM == 256) launch_kernel<16, 2>(grid, stream, map_a, map_b, p);
    else if (TM == 128) launch_kernel<8, 2>(grid, stream, map_a, map_b, p);
    else launch_kernel<4, 2>(grid, stream, map_a, map_b, p);
  } else {
    if (TM == 256) launch_kernel<16, 1>(grid, stream, map_a, map_b, p);
    else if (TM == 128) launch_kernel<8, 1>(grid, stream, map_a, map_b, p);
    else launch_kernel<4, 1>(grid, stream, map_a, map_b, p);
  }
  if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  if (p.tail_tiles > 0 && p.tail_ipc < p.kblocks) {
    launch_pdl(sgemm_tail_reduce_kernel, dim3(p.tail_tiles, 16), dim3(256), 0, stream, p);
    if (cudaGetLastError() != cudaSuccess) return DGEMM_ERR_CUDA;
  }
  return DGEMM_OK;
}

}  // namespace

extern "C" {

int sgemm_f32(int64_t M, int64_t N, int64_t K, const float* A, int64_t lda, const float* B, int64_t ldb, float* C,
              int64_t ldc, void* stream) {
  const int v = validate(M, N, K, A, lda, B, ldb, C, ldc);
  if (v == 1) return DGEMM_OK;
  if (v != DGEMM_OK) return v;
  return launch(M, N, K, A, lda, B, ldb, C, ldc, static_cast<cudaStream_t>(stream));
}

int sgemm_last_device_status(void* stream) {
  DeviceState* st = nullptr;
  const int rc = device_state(&st);
  if (rc != DGEMM_OK) return rc;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
    (void)cudaGetLastError();
    return DGEMM_ERR_CUDA;
  }
  int v = 0;
  if (cudaMemcpy(&v, st->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return DGEMM_ERR_CUDA;
  if (v != 0 && cudaMemset(st->status, 0, sizeof(int)) != cudaSuccess) return DGEMM_ERR_CUDA;
  return v;
}

}  // extern "C"
