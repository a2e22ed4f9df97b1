"""B200-native FP64 GEMM ``C += A @ B`` (row-major) behind the C ABI of ``libdgemm``.

The Python layer only marshals arguments; every step of the computation runs in the CUDA
kernels of ``csrc/``. The library is loaded lazily on first use and its absence is an error.
"""
from .binding import (  # noqa: F401
    DGEMM_OK,
    DGEMM_OP_N,
    DGEMM_OP_T,
    DGEMM_VARIANT_AUTO,
    DGEMM_VARIANT_GENERIC,
    DGEMM_VARIANT_NAIVE,
    DGEMM_VARIANT_TMA,
    DGEMM_VARIANT_TMA_WS,
    DGEMM_VARIANT_GENERIC_WS,
    DgemmError,
    dgemm_f64,
    dgemm_f64_ex,
    dgemm_f64_host,
    dgemm_f64_raw,
    dgemm_f64_static_ws,
    dgemm_fp64_peak_probe,
    dgemm_last_device_status,
    dgemm_launch_count,
    dgemm_plan,
    dgemm_selftest_wait_timeout,
    dgemm_set_split_k,
    dgemm_set_test_flags,
    dgemm_set_variant,
    dgemm_strerror,
    dgemm_version,
    lib_path,
    load_library,
    sgemm_f32,
    sgemm_last_device_status,
)
