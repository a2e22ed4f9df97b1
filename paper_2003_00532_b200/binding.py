"""ctypes binding of ``libdgemm.so``: same names as the C ABI in ``include/dgemm.h``.

Argument marshalling only. Matrices are passed as 2-D float64 ``torch`` tensors with unit
column stride (the row stride is the leading dimension, so a view ``buf[:, :cols]`` of a wider
buffer expresses padding) or as raw integer addresses with explicit sizes. There is no CPU or
library fallback: if the shared library is missing, loading fails with an error.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libdgemm.so")
_lock = threading.Lock()
_lib: Optional[ctypes.CDLL] = None

DGEMM_OK = 0
DGEMM_ERR_BAD_DIM = -1
DGEMM_ERR_BAD_LD = -2
DGEMM_ERR_NULL = -3
DGEMM_ERR_ALIGN = -4
DGEMM_ERR_ALIAS = -5
DGEMM_ERR_DEVICE = -6
DGEMM_ERR_CUDA = -7
DGEMM_ERR_TIMEOUT = -8
DGEMM_ERR_VARIANT = -9
DGEMM_ERR_SIZE = -10

DGEMM_OP_N = 0
DGEMM_OP_T = 1

DGEMM_VARIANT_AUTO = -1
DGEMM_VARIANT_NAIVE = 0
DGEMM_VARIANT_TMA = 1
DGEMM_VARIANT_GENERIC = 2
DGEMM_VARIANT_TMA_WS = 3
DGEMM_VARIANT_GENERIC_WS = 4
DGEMM_VARIANT_TMA_CLUSTER = 5
DGEMM_VARIANT_GENERIC_CLUSTER = 6
DGEMM_VARIANT_SMEM = 7
DGEMM_VARIANT_TMA_DFMA = 8
DGEMM_VARIANT_GENERIC_DFMA = 9
DGEMM_VARIANT_TMA_WS_BULK = 10

# dgemm_set_test_flags bits
DGEMM_TEST_NO_C_PREFETCH = 1
DGEMM_TEST_NO_BLOCKED_B = 2
DGEMM_TEST_TALL_TILES = 4
DGEMM_TEST_SMALL_WARP_TILES = 8
DGEMM_TEST_NO_PACKING = 16
DGEMM_TEST_WS_TWO_CTAS = 32
DGEMM_TEST_NO_CLUSTER = 128
DGEMM_TEST_DROP_LOADS = 256


class DgemmError(RuntimeError):
    """A libdgemm call returned a negative status."""

    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dgemm_strerror(status)} (status {status})")


def lib_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Load ``libdgemm.so`` (built in-tree by ``build.py``). Raises if it is absent."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(_LIB_PATH):
                raise FileNotFoundError(
                    f"{_LIB_PATH} not found: build it with `python -m paper_2003_00532_b200.build` "
                    "(nvcc, sm_100a); there is no fallback path")
            lib = ctypes.CDLL(_LIB_PATH)
            i64, vp = ctypes.c_int64, ctypes.c_void_p
            lib.dgemm_f64.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, vp]
            lib.dgemm_f64.restype = ctypes.c_int
            lib.dgemm_f64_host.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64]
            lib.dgemm_f64_host.restype = ctypes.c_int
            lib.dgemm_f64_ex.argtypes = [ctypes.c_int, ctypes.c_int, i64, i64, i64, ctypes.c_double, vp, i64, vp, i64,
                                         ctypes.c_double, vp, i64, vp]
            lib.dgemm_f64_ex.restype = ctypes.c_int
            lib.sgemm_f32.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, vp]
            lib.sgemm_f32.restype = ctypes.c_int
            lib.sgemm_last_device_status.argtypes = [vp]
            lib.sgemm_last_device_status.restype = ctypes.c_int
            lib.dgemm_plan.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
            lib.dgemm_plan.restype = ctypes.c_int
            lib.dgemm_f64_static_ws.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, ctypes.c_int, vp]
            lib.dgemm_f64_static_ws.restype = ctypes.c_int
            lib.dgemm_strerror.argtypes = [ctypes.c_int]
            lib.dgemm_strerror.restype = ctypes.c_char_p
            lib.dgemm_version.argtypes = []
            lib.dgemm_version.restype = ctypes.c_int
            lib.dgemm_set_variant.argtypes = [ctypes.c_int]
            lib.dgemm_set_variant.restype = ctypes.c_int
            lib.dgemm_set_test_flags.argtypes = [ctypes.c_int]
            lib.dgemm_set_test_flags.restype = ctypes.c_int
            lib.dgemm_set_split_k.argtypes = [ctypes.c_int]
            lib.dgemm_set_split_k.restype = ctypes.c_int
            lib.dgemm_last_device_status.argtypes = [vp]
            lib.dgemm_last_device_status.restype = ctypes.c_int
            lib.dgemm_selftest_wait_timeout.argtypes = [ctypes.c_int]
            lib.dgemm_selftest_wait_timeout.restype = ctypes.c_int
            lib.dgemm_release_scratch.argtypes = []
            lib.dgemm_release_scratch.restype = ctypes.c_int
            lib.dgemm_launch_count.argtypes = []
            lib.dgemm_launch_count.restype = ctypes.c_int64
            lib.dgemm_fp64_peak_probe.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                                  ctypes.POINTER(ctypes.c_double)]
            lib.dgemm_fp64_peak_probe.restype = ctypes.c_int
            lib.dgemm_fp64_fma_probe.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                                 ctypes.POINTER(ctypes.c_double)]
            lib.dgemm_fp64_fma_probe.restype = ctypes.c_int
            _lib = lib
    return _lib


def _matrix_args(x, name: str, want_cuda: bool, dtype=None):
    """(address, rows, cols, ld) of a 2-D float64 (or `dtype`) tensor with unit column stride."""
    import torch
    dtype = dtype or torch.float64
    if not isinstance(x, torch.Tensor):
        raise TypeError(f"{name}: expected a torch.Tensor")
    if x.dtype != dtype or x.dim() != 2:
        raise TypeError(f"{name}: need a 2-D {str(dtype).replace('torch.', '')} tensor")
    if x.is_cuda != want_cuda:
        raise ValueError(f"{name}: expected a {'CUDA' if want_cuda else 'host'} tensor")
    rows, cols = x.shape
    if rows > 0 and cols > 0 and x.stride(1) != 1:
        raise ValueError(f"{name}: columns must be contiguous (row-major)")
    ld = max(cols, 1)
    if rows >= 1 and cols > 0 and x.stride(0) >= ld:
        ld = x.stride(0)  # a one-row view keeps its buffer's leading dimension
    return x.data_ptr(), rows, cols, ld


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _shapes(A, B, C, cuda: bool):
    pa, M, K, lda = _matrix_args(A, "A", cuda)
    pb, K2, N, ldb = _matrix_args(B, "B", cuda)
    pc, M2, N2, ldc = _matrix_args(C, "C", cuda)
    if K != K2 or M != M2 or N != N2:
        raise ValueError(f"shape mismatch: A {tuple(A.shape)}, B {tuple(B.shape)}, C {tuple(C.shape)}")
    return M, N, K, pa, lda, pb, ldb, pc, ldc


def dgemm_f64(A, B, C, stream=None, check: bool = True) -> int:
    """``C += A @ B`` on the current CUDA device, asynchronously on ``stream``.

    ``A`` (M x K), ``B`` (K x N), ``C`` (M x N): CUDA float64 tensors, row-major, row stride =
    leading dimension. ``stream``: a ``torch.cuda.Stream``, a raw ``cudaStream_t`` integer, or
    ``None`` for torch's current stream. Returns the status; raises ``DgemmError`` on a negative
    status unless ``check=False``.
    """
    M, N, K, pa, lda, pb, ldb, pc, ldc = _shapes(A, B, C, True)
    return dgemm_f64_raw(M, N, K, pa, lda, pb, ldb, pc, ldc, _stream_handle(stream), check)


def dgemm_f64_raw(M, N, K, A_ptr, lda, B_ptr, ldb, C_ptr, ldc, stream: Optional[int] = None,
                  check: bool = True) -> int:
    """The C entry point with raw addresses (device pointers as integers)."""
    rc = load_library().dgemm_f64(M, N, K, A_ptr, lda, B_ptr, ldb, C_ptr, ldc, stream)
    if check and rc < 0:
        raise DgemmError(rc, "dgemm_f64")
    return rc


def dgemm_f64_ex(A, B, C, alpha: float = 1.0, beta: float = 1.0, transa: bool = False, transb: bool = False,
                 stream=None, check: bool = True) -> int:
    """``C = alpha * op(A) @ op(B) + beta * C`` on the current CUDA device, asynchronously.

    ``A`` and ``B`` are passed as stored: ``A`` is K x M when ``transa`` (used as its transpose),
    ``B`` is N x K when ``transb``. ``beta == 0`` never reads ``C``; ``alpha == 0`` never reads
    ``A`` or ``B``. Otherwise as :func:`dgemm_f64`.
    """
    pa, ar, ac, lda = _matrix_args(A, "A", True)
    pb, br, bc, ldb = _matrix_args(B, "B", True)
    pc, M, N, ldc = _matrix_args(C, "C", True)
    Ma, K = (ac, ar) if transa else (ar, ac)
    K2, Nb = (bc, br) if transb else (br, bc)
    if K != K2 or Ma != M or Nb != N:
        raise ValueError(f"shape mismatch: A {tuple(A.shape)} (transa={transa}), B {tuple(B.shape)} "
                         f"(transb={transb}), C {tuple(C.shape)}")
    rc = load_library().dgemm_f64_ex(DGEMM_OP_T if transa else DGEMM_OP_N, DGEMM_OP_T if transb else DGEMM_OP_N,
                                     M, N, K, float(alpha), pa, lda, pb, ldb, float(beta), pc, ldc,
                                     _stream_handle(stream))
    if check and rc < 0:
        raise DgemmError(rc, "dgemm_f64_ex")
    return rc


def sgemm_f32(A, B, C, stream=None, check: bool = True) -> int:
    """Single precision ``C += A @ B`` (CUDA float32 tensors, row-major, row stride = leading
    dimension), exact binary32 arithmetic, asynchronously on ``stream``."""
    import torch
    pa, M, K, lda = _matrix_args(A, "A", True, torch.float32)
    pb, K2, N, ldb = _matrix_args(B, "B", True, torch.float32)
    pc, M2, N2, ldc = _matrix_args(C, "C", True, torch.float32)
    if K != K2 or M != M2 or N != N2:
        raise ValueError(f"shape mismatch: A {tuple(A.shape)}, B {tuple(B.shape)}, C {tuple(C.shape)}")
    rc = load_library().sgemm_f32(M, N, K, pa, lda, pb, ldb, pc, ldc, _stream_handle(stream))
    if check and rc < 0:
        raise DgemmError(rc, "sgemm_f32")
    return rc


def sgemm_last_device_status(stream=None) -> int:
    return int(load_library().sgemm_last_device_status(_stream_handle(stream)))


def dgemm_f64_static_ws(A, B, C, split_k: int = 0, stream=None, check: bool = True) -> int:
    """``C += A @ B`` with split-K partial sums kept in the library's fixed device array.

    For callers that may not allocate device memory when they call (under a lock shared with an
    allocator, under a fixed memory budget, in a latency-critical loop): this entry point never
    allocates. At most 128 partial tiles (``ceil(M/128) * ceil(N/128) * split_k``); beyond that it
    returns ``DGEMM_ERR_SIZE``. Calls on one device share the array, so they must not overlap on
    the GPU. The first call on a device does the set-up and should come before any stream capture.
    """
    M, N, K, pa, lda, pb, ldb, pc, ldc = _shapes(A, B, C, True)
    rc = load_library().dgemm_f64_static_ws(M, N, K, pa, lda, pb, ldb, pc, ldc, int(split_k),
                                            _stream_handle(stream))
    if check and rc < 0:
        raise DgemmError(rc, "dgemm_f64_static_ws")
    return rc


def dgemm_f64_host(A, B, C, check: bool = True) -> int:
    """``C += A @ B`` with HOST tensors: the library copies to the device, computes there and
    copies the result back into ``C``. Synchronous."""
    M, N, K, pa, lda, pb, ldb, pc, ldc = _shapes(A, B, C, False)
    rc = load_library().dgemm_f64_host(M, N, K, pa, lda, pb, ldb, pc, ldc)
    if check and rc < 0:
        raise DgemmError(rc, "dgemm_f64_host")
    return rc


PLAN_FIELDS = ("variant", "bm", "bn", "wtm", "ctas_per_sm", "grid", "kblocks", "split_k", "kblocks_per_split",
               "dp_tiles", "tail_tiles", "tail_ipc")


def dgemm_plan(M: int, N: int, K: int, tma_addressable: bool = True, sm_count: int = 0) -> dict:
    """The kernel, tile and work decomposition ``dgemm_f64`` would use for this shape under the
    current settings (host logic only; needs no GPU)."""
    out = (ctypes.c_int * 12)()
    rc = load_library().dgemm_plan(int(M), int(N), int(K), int(bool(tma_addressable)), int(sm_count), out)
    if rc < 0:
        raise DgemmError(rc, "dgemm_plan")
    return dict(zip(PLAN_FIELDS, (int(v) for v in out)))


def dgemm_strerror(status: int) -> str:
    return load_library().dgemm_strerror(int(status)).decode()


def dgemm_version() -> int:
    return int(load_library().dgemm_version())


def dgemm_set_variant(variant: int) -> int:
    rc = load_library().dgemm_set_variant(int(variant))
    if rc < 0:
        raise DgemmError(rc, "dgemm_set_variant")
    return rc


def dgemm_set_split_k(split_k: int) -> int:
    rc = load_library().dgemm_set_split_k(int(split_k))
    if rc < 0:
        raise DgemmError(rc, "dgemm_set_split_k")
    return rc


def dgemm_set_test_wait_limit(limit_us: int) -> int:
    """Testing aid: limit of the kernels' main-loop waits in microseconds (0 = the default four seconds)."""
    rc = load_library().dgemm_set_test_wait_limit(int(limit_us))
    if rc < 0:
        raise DgemmError(rc, "dgemm_set_test_wait_limit")
    return rc


def dgemm_set_test_flags(flags: int) -> int:
    """Testing aid (bits): 1 no L2 prefetch of C, 2 no single-copy staging of B, 4 128-row tiles,
    8 32 x 32 warp tiles, 16 no packing pass, 32 two-CTA form of the warp-specialised kernel."""
    rc = load_library().dgemm_set_test_flags(int(flags))
    if rc < 0:
        raise DgemmError(rc, "dgemm_set_test_flags")
    return rc


def dgemm_last_device_status(stream=None) -> int:
    return int(load_library().dgemm_last_device_status(_stream_handle(stream)))


def dgemm_selftest_wait_timeout(limit_us: int = 1000) -> int:
    """Runs the bounded-wait self-test (a wait that must give up after ``limit_us``)."""
    rc = load_library().dgemm_selftest_wait_timeout(int(limit_us))
    if rc < 0:
        raise DgemmError(rc, "dgemm_selftest_wait_timeout")
    return rc


def dgemm_launch_count() -> int:
    return int(load_library().dgemm_launch_count())


def dgemm_release_scratch() -> int:
    """Frees the library's device scratch on the current device (it comes back on demand)."""
    rc = load_library().dgemm_release_scratch()
    if rc < 0:
        raise DgemmError(rc, "dgemm_release_scratch")
    return rc


def dgemm_fp64_peak_probe(millis: int = 200):
    """Returns ``(fma_per_clk_sm, tflops)`` measured by the register-only DMMA loop."""
    a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = load_library().dgemm_fp64_peak_probe(int(millis), ctypes.byref(a), ctypes.byref(b))
    if rc < 0:
        raise DgemmError(rc, "dgemm_fp64_peak_probe")
    return a.value, b.value


def dgemm_fp64_fma_probe(millis: int = 200):
    """Returns ``(fma_per_clk_sm, tflops)`` measured by the register-only loop of plain FP64 FMAs."""
    a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = load_library().dgemm_fp64_fma_probe(int(millis), ctypes.byref(a), ctypes.byref(b))
    if rc < 0:
        raise DgemmError(rc, "dgemm_fp64_fma_probe")
    return a.value, b.value
