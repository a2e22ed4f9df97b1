"""The warp-specialised kernel whose epilogue leaves through the copy engine (bulk reduce into C row by row,
or bulk store for beta == 0), forced on shapes of every kind and as the library's own choice on
rank-k updates. Needs a B200. Everything is compared with the CPU oracle: bit for bit on
integer-valued data, within the bound of the other parity tests on real data."""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl
from test_gpu_parity import _check_full, run_gpu

pytestmark = pytest.mark.gpu

BULK = dg.DGEMM_VARIANT_TMA_WS_BULK

# ragged in every dimension: rows beyond M are not sent, the tiles of a ragged last tile column are
# added to C by the arithmetic warps themselves
SHAPES = [(1, 2, 1), (17, 14, 11), (127, 130, 47), (128, 128, 16), (129, 126, 17), (130, 260, 33), (257, 132, 100),
          (200, 300, 1), (1000, 32, 600), (513, 34, 64), (1000, 1538, 777), (640, 384, 2048), (2304, 2304, 64)]


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", SHAPES)
def test_forced_bulk_epilogue(oracle, shape, integer):
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=500 + M + N + K, lda=K + 2 + (K & 1), ldb=N + 4 + (N & 1), ldc=N + 6,
                           integer=integer)
    _check_full(oracle, prob, run_gpu(prob, BULK))


@pytest.mark.parametrize("split", [2, 7])
def test_bulk_epilogue_with_partial_tiles(oracle, split):
    """Forced split K: partial tiles go to the workspace and the reduction kernel, as in the other kernels."""
    prob = wl.make_problem(200, 150, 1000, seed=11, lda=1000, ldb=152, ldc=152, integer=True)
    _check_full(oracle, prob, run_gpu(prob, BULK, split_k=split))


def test_bulk_epilogue_refuses_a_c_the_copy_engine_cannot_address():
    A = torch.zeros(64, 64, dtype=torch.float64, device="cuda")
    Cbuf = torch.zeros(64 * 65 + 1, dtype=torch.float64, device="cuda")
    dg.dgemm_set_variant(BULK)
    try:
        odd_ld = Cbuf[:64 * 65].view(64, 65)[:, :64]
        assert dg.dgemm_f64(A, A, odd_ld, check=False) == dg.binding.DGEMM_ERR_VARIANT
        off = Cbuf[1:1 + 64 * 64].view(64, 64)   # base 8 bytes off a 16-byte boundary
        assert dg.dgemm_f64(A, A, off, check=False) == dg.binding.DGEMM_ERR_VARIANT
        assert dg.dgemm_f64_ex(A, A, Cbuf[:4096].view(64, 64), alpha=1.0, beta=0.5, check=False) == dg.binding.DGEMM_ERR_VARIANT
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    assert dg.dgemm_last_device_status() == 0


@pytest.mark.parametrize("alpha,beta", [(1.0, 0.0), (-2.5, 1.0), (3.0, 0.0)])
def test_bulk_epilogue_general_form(oracle, alpha, beta):
    """beta == 0 stores without ever reading C (NaN in the old C does not survive); alpha scales the product."""
    rng = np.random.Generator(np.random.PCG64(5))
    M, N, K = 300, 258, 190
    a = rng.integers(-4, 5, (M, K)).astype(np.float64)
    b = rng.integers(-4, 5, (K, N)).astype(np.float64)
    c = rng.integers(-4, 5, (M, N)).astype(np.float64)
    if beta == 0.0:
        c[5, 7] = np.nan
        c[200, 257] = np.inf
    dC = torch.from_numpy(c).cuda()
    dg.dgemm_set_variant(BULK)
    try:
        dg.dgemm_f64_ex(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda(), dC, alpha=alpha, beta=beta)
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    assert dg.dgemm_last_device_status() == 0
    want = c.copy()
    oracle.dgemm_oracle_general(False, False, alpha, a, b, beta, want)
    assert np.array_equal(dC.cpu().numpy(), want)


def test_auto_picks_the_bulk_epilogue_for_rank_k_updates(oracle):
    """A large problem with a short K and an addressable C runs the bulk-epilogue kernel by the library's
    own choice; with an odd ldc it does not. Both are right."""
    plan = dg.dgemm_plan(16384, 16384, 64)
    assert plan["variant"] == BULK
    for ldc in (4096, 4097):
        prob = wl.make_problem(4096, 4096, 64, seed=9, ldc=ldc, integer=True)
        out = run_gpu(prob)
        _check_full(oracle, prob, out)
