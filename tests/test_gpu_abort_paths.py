"""The abort paths inside the GEMM kernels, exercised without a fault. Needs a B200.

Failure is injected from the host: with DGEMM_TEST_DROP_LOADS the kernels' producers skip their copies,
so the stage barriers the arithmetic waits on are never completed, and dgemm_set_test_wait_limit
shortens the main-loop waits to a few milliseconds. Every kernel family must then give up its waits,
record DGEMM_ERR_TIMEOUT in the device status word, let all of its warps (and, in the cluster kernel,
all thread blocks of the cluster) reach the closing barriers and return normally; the context stays
usable and the next call is correct. Nothing traps, faults or spins without a limit.
"""
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl
from test_gpu_parity import _check_full, run_gpu

pytestmark = pytest.mark.gpu

TIMEOUT = dg.binding.DGEMM_ERR_TIMEOUT

# (variant, flags, shape, odd leading dimensions): one small problem per kernel and staging
CASES = [
    (dg.DGEMM_VARIANT_TMA, 0, (300, 260, 200), False),              # inline kernel, 64 x 128 tiles, TMA staging
    (dg.DGEMM_VARIANT_TMA, dg.DGEMM_TEST_TALL_TILES, (300, 260, 200), False),  # 128 x 128 tiles
    (dg.DGEMM_VARIANT_GENERIC, 0, (300, 260, 200), True),           # inline kernel, 8-byte asynchronous copies
    (dg.DGEMM_VARIANT_TMA_WS, 0, (300, 260, 2000), False),          # warp-specialised, 128 x 128
    (dg.DGEMM_VARIANT_TMA_WS, dg.DGEMM_TEST_WS_TWO_CTAS, (300, 260, 200), False),  # warp-specialised, 64 x 128, two CTAs per SM
    (dg.DGEMM_VARIANT_GENERIC_WS, 0, (300, 260, 200), True),        # warp-specialised, generic staging
    (dg.DGEMM_VARIANT_TMA_CLUSTER, 0, (200, 300, 400), False),      # clusters: every CTA still reaches both cluster barriers
    (dg.DGEMM_VARIANT_GENERIC_CLUSTER, 0, (200, 300, 400), True),
    (dg.DGEMM_VARIANT_TMA_WS_BULK, 0, (300, 260, 200), False),      # bulk epilogue: the hand-over warp gives up as well
    (dg.DGEMM_VARIANT_TMA_DFMA, 0, (300, 260, 200), False),
    (dg.DGEMM_VARIANT_AUTO, 0, (1024, 1024, 1024), False),          # the library's own choice, partial tiles and reduction kernel behind it
]


@pytest.mark.parametrize("variant,flags,shape,odd", CASES)
def test_dropped_loads_end_in_a_reported_timeout(oracle, variant, flags, shape, odd):
    M, N, K = shape
    ld = dict(lda=K + 3, ldb=N + 5, ldc=N + 7) if odd else dict(lda=K + 2 + (K & 1), ldb=N + 4 + (N & 1), ldc=N + 6)
    prob = wl.make_problem(M, N, K, seed=7, integer=True, **ld)
    A, B, C = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    assert dg.dgemm_last_device_status() == dg.DGEMM_OK
    dg.dgemm_set_variant(variant)
    dg.dgemm_set_test_wait_limit(3000)  # 3 ms
    dg.dgemm_set_test_flags(flags | dg.DGEMM_TEST_DROP_LOADS)
    try:
        rc = dg.dgemm_f64(A[:, :K], B[:, :N], C[:, :N])    # launches fine: the failure is on the device
        assert rc == dg.DGEMM_OK
        assert dg.dgemm_last_device_status() == TIMEOUT    # synchronises: the kernels have returned
        assert dg.dgemm_last_device_status() == dg.DGEMM_OK  # read and cleared
    finally:
        dg.dgemm_set_test_flags(0)
        dg.dgemm_set_test_wait_limit(0)
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    # the same kernel, undisturbed, right afterwards
    dg.dgemm_set_test_flags(flags)
    try:
        out = run_gpu(prob, variant)
    finally:
        dg.dgemm_set_test_flags(0)
    _check_full(oracle, prob, out)


def test_wait_limit_setter_rejects_nonsense():
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_test_wait_limit(-1)
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_test_wait_limit(5000000)
    assert dg.dgemm_set_test_wait_limit(0) == 0
