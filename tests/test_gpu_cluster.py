"""Parity of the cluster split-K kernel (DGEMM_VARIANT_TMA_CLUSTER: K cut over the CTAs of a
thread-block cluster, partial tiles added through distributed shared memory) against the CPU
oracle, and its bit-identity with the workspace split of the same K partition. Needs a B200.

Same bars as the other parity tests: bit-exact on integer-valued inputs, the K-term rounding bound
on real inputs.
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from test_gpu_general import _case, _draw, _padded_dev, _rng

pytestmark = pytest.mark.gpu

V_CLUSTER = dg.DGEMM_VARIANT_TMA_CLUSTER


@pytest.mark.parametrize("split", [0, 1, 2, 4, 8])
@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", [
    (64, 128, 16),      # one tile, one k-block: with 2, 4, 8 CTAs all ranks but the first idle
    (1, 2, 2),
    (65, 130, 18),      # ragged in M, N and K
    (128, 128, 128),
    (250, 134, 90),
    (100, 200, 300),
    (300, 1000, 78),    # 40 tiles: several clusters per GPC
    (512, 512, 512),
    (1000, 1000, 200),  # 128 tiles x 8 CTAs: more clusters than fit at once
])
def test_cluster_kernel_forced(oracle, shape, integer, split):
    M, N, K = shape
    _case(oracle, M, N, K, False, False, 1.0, 1.0, integer, seed=M + 7 * N + 13 * K + split,
          variant=V_CLUSTER, split_k=split)


@pytest.mark.parametrize("split", [2, 8])
@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("alpha,beta", [(2.0, -3.0), (0.375, 0.0), (-1.0, 0.5), (1.0, 0.0)])
@pytest.mark.parametrize("ta,tb", [(False, False), (True, False), (False, True), (True, True)])
def test_cluster_kernel_general_form(oracle, ta, tb, alpha, beta, integer, split):
    # padded leading dimensions (kept even: the forced variant needs operands TMA can address;
    # transposed operands are rewritten into aligned scratch first), odd ldc
    _case(oracle, 190, 200, 150, ta, tb, alpha, beta, integer, seed=91 + split, pad=(2, 4, 7),
          variant=V_CLUSTER, split_k=split)


def test_cluster_kernel_beta_zero_ignores_old_c(oracle):
    # beta == 0: C is write-only, NaN and Inf in it must not reach the result
    _case(oracle, 130, 140, 100, False, False, 1.5, 0.0, False, seed=5, c_fill=float("nan"),
          variant=V_CLUSTER, split_k=4)
    _case(oracle, 130, 140, 100, False, False, 1.0, 0.0, True, seed=6, c_fill=float("inf"),
          variant=V_CLUSTER, split_k=8)


def test_cluster_kernel_sign_of_zero(oracle):
    # all-zero products: the sum of the partial tiles must keep IEEE signs (-0 + -0 = -0, and an
    # idle rank must not contribute a +0)
    M, N, K = 64, 128, 32
    A = np.zeros((M, K))
    B = np.ones((K, N))
    A[::2] = -0.0
    for split in (2, 8):
        C = np.full((M, N), -0.0)
        want = C.copy()
        oracle.dgemm_oracle_general(False, False, 1.0, A, B, 1.0, want)
        dA, dB, dC = (torch.from_numpy(x).cuda() for x in (A, B, C))
        dg.dgemm_set_variant(V_CLUSTER)
        dg.dgemm_set_split_k(split)
        try:
            dg.dgemm_f64(dA, dB, dC)
        finally:
            dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
            dg.dgemm_set_split_k(0)
        assert dC.cpu().numpy().tobytes() == want.tobytes()


@pytest.mark.parametrize("shape,split", [((128, 128, 128), 8), ((200, 300, 400), 4), ((512, 512, 512), 4),
                                         ((190, 260, 1000), 2), ((64, 128, 4096), 8)])
def test_cluster_split_equals_workspace_split_bit_for_bit(shape, split):
    """The same K partition through the workspace and a second kernel (uniform split-K of the
    inline kernel) gives the same bits: both add the partial tiles in partition order."""
    M, N, K = shape
    rng = _rng(M + N + K)
    A, B, C = _draw(rng, (M, K), False), _draw(rng, (K, N), False), _draw(rng, (M, N), False)
    out = []
    for variant in (V_CLUSTER, dg.DGEMM_VARIANT_TMA):
        _, dA = _padded_dev(A, K)
        _, dB = _padded_dev(B, N)
        _, dC = _padded_dev(C, N)
        dg.dgemm_set_variant(variant)
        dg.dgemm_set_split_k(split)
        try:
            dg.dgemm_f64(dA, dB, dC)
            assert dg.dgemm_last_device_status() == dg.DGEMM_OK
        finally:
            dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
            dg.dgemm_set_split_k(0)
        out.append(dC.cpu().numpy().copy())
    assert out[0].tobytes() == out[1].tobytes()


@pytest.mark.parametrize("shape", [(32, 32, 32), (64, 64, 64), (192, 192, 192), (128, 80, 32), (48, 480, 48),
                                   (320, 320, 320), (512, 512, 256), (1936, 240, 96), (558, 26, 26)])
@pytest.mark.parametrize("integer", [True, False])
def test_auto_picks_cluster_kernel_on_small_problems(oracle, shape, integer):
    """What DGEMM_VARIANT_AUTO does below one wave of tiles: one launch of the cluster kernel. The
    same shapes with the cluster kernel switched off take the general kernels; both match the oracle."""
    M, N, K = shape
    pl = dg.dgemm_plan(M, N, K)
    assert pl["variant"] == V_CLUSTER and pl["bm"] == 64 and pl["bn"] == 128, pl
    assert pl["grid"] == pl["split_k"] * pl["dp_tiles"] and pl["split_k"] in (2, 4, 8)
    n0 = dg.dgemm_launch_count()
    _case(oracle, M, N, K, False, False, 1.0, 1.0, integer, seed=3 * M + N + K)
    assert dg.dgemm_launch_count() - n0 == 1
    dg.dgemm_set_test_flags(dg.DGEMM_TEST_NO_CLUSTER)
    try:
        assert dg.dgemm_plan(M, N, K)["variant"] != V_CLUSTER
        _case(oracle, M, N, K, False, False, 1.0, 1.0, integer, seed=3 * M + N + K)
    finally:
        dg.dgemm_set_test_flags(0)


@pytest.mark.parametrize("split", [0, 2, 8])
@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", [(65, 129, 17), (282, 85, 44), (250, 133, 91), (300, 1001, 77), (21, 97, 75)])
def test_cluster_kernel_generic_staging(oracle, shape, integer, split):
    """Odd leading dimensions and bases off the 16-byte boundary: 8-byte asynchronous copies instead
    of TMA, everything else the same kernel. Forced, and as DGEMM_VARIANT_AUTO picks it."""
    M, N, K = shape
    _case(oracle, M, N, K, False, False, 1.0, 1.0, integer, seed=M + N + K + split, pad=(1, 3, 1), offset=1,
          variant=dg.DGEMM_VARIANT_GENERIC_CLUSTER, split_k=split)
    if split == 0:
        _case(oracle, M, N, K, False, False, -2.0, 0.5, integer, seed=M + N + K, pad=(1, 3, 1), offset=1)


def test_auto_picks_generic_cluster_kernel_for_small_unaddressable_problems():
    for shape in [(282, 85, 44), (21, 97, 75), (64, 64, 64)]:
        assert dg.dgemm_plan(*shape, tma_addressable=False)["variant"] == dg.DGEMM_VARIANT_GENERIC_CLUSTER


def test_forced_cluster_variant_rejects_operands_tma_cannot_address():
    A = torch.zeros(64, 33, dtype=torch.float64, device="cuda")  # odd leading dimension
    B = torch.zeros(33, 128, dtype=torch.float64, device="cuda")
    C = torch.zeros(64, 128, dtype=torch.float64, device="cuda")
    dg.dgemm_set_variant(V_CLUSTER)
    try:
        rc = dg.load_library().dgemm_f64(64, 128, 33, A.data_ptr(), 33, B.data_ptr(), 128, C.data_ptr(), 128, None)
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    assert rc == dg.DGEMM_ERR_VARIANT
