"""Parity of the general entry point ``C = alpha * op(A) op(B) + beta * C`` against the CPU oracle's
definition of it. Needs a B200.

Bit-exact on integer-valued inputs with integer scalars; on uniform real inputs
|dC_ij| <= 2 (K+3) 2^-53 (|alpha| |A||B| + |beta| |C|)_ij: each side accumulates K products, then
rounds once for alpha, once (fused or not) for beta*C and the add.
"""
import itertools

import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg

pytestmark = pytest.mark.gpu

U = 2.0 ** -53
FORMS = list(itertools.product([False, True], repeat=2))


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _draw(rng, shape, integer):
    if integer:
        return rng.integers(-4, 5, size=shape).astype(np.float64)
    return rng.uniform(-1.0, 1.0, size=shape)


def _padded_dev(x: np.ndarray, ld: int, offset: int = 0):
    """Device buffer of rows x ld doubles (NaN padding) starting `offset` doubles into an
    allocation; returns (buffer view rows x ld, logical view rows x cols)."""
    rows, cols = x.shape
    whole = torch.full((rows * ld + offset + 8,), float("nan"), dtype=torch.float64, device="cuda")
    buf = whole[offset:offset + rows * ld].view(rows, ld)
    buf[:, :cols] = torch.from_numpy(x).cuda()
    return buf, buf[:, :cols]


def _case(oracle, M, N, K, ta, tb, alpha, beta, integer, seed, pad=(0, 0, 0), offset=0, c_fill=None,
          variant=dg.DGEMM_VARIANT_AUTO, split_k=0):
    rng = _rng(seed)
    A = _draw(rng, (K, M) if ta else (M, K), integer)
    B = _draw(rng, (N, K) if tb else (K, N), integer)
    C = _draw(rng, (M, N), integer)
    if c_fill is not None:
        C[:] = c_fill
    _, dA = _padded_dev(A, A.shape[1] + pad[0], offset)
    _, dB = _padded_dev(B, B.shape[1] + pad[1], offset)
    bufC, dC = _padded_dev(C, N + pad[2], 0)
    dg.dgemm_set_variant(variant)
    dg.dgemm_set_split_k(split_k)
    try:
        dg.dgemm_f64_ex(dA, dB, dC, alpha=alpha, beta=beta, transa=ta, transb=tb)
        assert dg.dgemm_last_device_status() == dg.DGEMM_OK
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        dg.dgemm_set_split_k(0)
    got = dC.cpu().numpy()
    assert bool(torch.isnan(bufC[:, N:]).all()), "padding columns of C were modified"
    want = C.copy()
    oracle.dgemm_oracle_general(ta, tb, alpha, A, B, beta, want)
    if integer and float(alpha).is_integer() and float(beta).is_integer():
        assert np.ascontiguousarray(got).tobytes() == want.tobytes()
        return
    opA = A.T if ta else A
    opB = B.T if tb else B
    scale = abs(alpha) * (np.abs(opA) @ np.abs(opB)) + (abs(beta) * np.abs(C) if beta != 0.0 else 0.0)
    bound = 2.0 * (K + 3) * U * scale
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert (err <= bound).all(), f"max err/bound = {(err / np.maximum(bound, 1e-300)).max()}"


@pytest.mark.parametrize("ta,tb", FORMS)
@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("alpha,beta", [(1.0, 1.0), (2.0, -3.0), (0.375, 0.0), (-1.0, 0.5)])
def test_forms_and_scalars_ragged(oracle, ta, tb, integer, alpha, beta):
    """Several tiles in both directions with ragged edges, odd leading dimensions, all operand forms."""
    _case(oracle, 333, 257, 190, ta, tb, alpha, beta, integer, seed=1000 + 2 * ta + tb, pad=(3, 5, 7))


@pytest.mark.parametrize("ta,tb", FORMS)
def test_beta_zero_ignores_nan_in_c(oracle, ta, tb):
    """beta == 0: C is an output; NaN and Inf in its old contents must not survive. Covers the
    vector epilogue (aligned interior tiles), the edge epilogue and the partial-tile reduction."""
    _case(oracle, 384, 256, 512, ta, tb, 1.0, 0.0, True, seed=7, c_fill=np.nan)      # K split over CTAs
    _case(oracle, 1000, 520, 96, ta, tb, 2.0, 0.0, True, seed=8, c_fill=np.inf, pad=(0, 0, 3))


@pytest.mark.parametrize("alpha,beta", [(0.0, 2.0), (0.0, 0.0), (0.0, 1.0)])
def test_alpha_zero_never_reads_operands(oracle, alpha, beta):
    M, N, K = 300, 200, 64
    rng = _rng(3)
    C = _draw(rng, (M, N), True)
    if beta == 0.0:
        C[::3] = np.nan
    bufC, dC = _padded_dev(C, N + 3)
    bad = torch.full((M, K), float("nan"), dtype=torch.float64, device="cuda")
    bad_b = torch.full((K, N), float("nan"), dtype=torch.float64, device="cuda")
    dg.dgemm_f64_ex(bad, bad_b, dC, alpha=alpha, beta=beta)
    got = dC.cpu().numpy()
    want = np.zeros((M, N)) if beta == 0.0 else beta * C
    assert np.array_equal(got, want)
    assert bool(torch.isnan(bufC[:, N:]).all())


def test_k_zero_scales_c(oracle):
    M, N = 70, 45
    C = _draw(_rng(4), (M, N), True)
    bufC, dC = _padded_dev(C, N + 1)
    A = torch.zeros((M, 0), dtype=torch.float64, device="cuda")
    B = torch.zeros((0, N), dtype=torch.float64, device="cuda")
    dg.dgemm_f64_ex(A, B, dC, alpha=5.0, beta=-2.0)
    assert np.array_equal(dC.cpu().numpy(), -2.0 * C)
    assert bool(torch.isnan(bufC[:, N:]).all())


@pytest.mark.parametrize("shape", [(256, 256, 256), (2088, 2048, 2048), (513, 33, 64), (1000, 32, 600)])
def test_unit_scalars_match_plain_entry_bit_for_bit(shape):
    """alpha = beta = 1 without transposition is the paper's operation: same bits as dgemm_f64 on
    real data (same kernels, fma(c, 1, acc) rounds like c + acc)."""
    M, N, K = shape
    g = torch.Generator(device="cuda").manual_seed(5)
    A = torch.rand(M, K, dtype=torch.float64, device="cuda", generator=g) * 2 - 1
    B = torch.rand(K, N, dtype=torch.float64, device="cuda", generator=g) * 2 - 1
    C = torch.rand(M, N, dtype=torch.float64, device="cuda", generator=g) * 2 - 1
    C1, C2 = C.clone(), C.clone()
    dg.dgemm_f64(A, B, C1)
    dg.dgemm_f64_ex(A, B, C2, alpha=1.0, beta=1.0)
    assert torch.equal(C1.view(torch.int64), C2.view(torch.int64))


@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC, dg.DGEMM_VARIANT_TMA_WS,
                                     dg.DGEMM_VARIANT_GENERIC_WS])
@pytest.mark.parametrize("split_k", [0, 3])
def test_every_pipeline_variant_applies_the_scalars(oracle, variant, split_k):
    """The scalars live in the shared epilogue and in the partial-tile reductions: every pipeline
    variant, with and without a forced K split, real and integer data, transposed B."""
    _case(oracle, 640, 384, 320, False, True, -2.0, 3.0, True, seed=21, variant=variant, split_k=split_k)
    _case(oracle, 640, 384, 320, True, False, 0.7, -1.3, False, seed=22, variant=variant, split_k=split_k)


def test_naive_variant_refuses_scalars():
    A = torch.zeros(8, 8, dtype=torch.float64, device="cuda")
    C = torch.zeros(8, 8, dtype=torch.float64, device="cuda")
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_NAIVE)
    try:
        assert dg.dgemm_f64_ex(A, A.clone(), C, alpha=2.0, check=False) == dg.binding.DGEMM_ERR_VARIANT
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)


@pytest.mark.parametrize("ta,tb", FORMS)
def test_narrow_and_unaligned(oracle, ta, tb):
    """N <= 32 (narrow tile) and operands that start 8 bytes off a 16-byte boundary."""
    _case(oracle, 1000, 31, 333, ta, tb, 1.5, -0.5, False, seed=31, pad=(1, 1, 1), offset=1)
    _case(oracle, 200, 130, 77, ta, tb, 2.0, 1.0, True, seed=32, pad=(1, 2, 0), offset=1)


@pytest.mark.parametrize("ta,tb", FORMS)
def test_large_forms_sampled(oracle, ta, tb):
    """2088 x 2048 x 2048 (the paper's problem size) in every operand form: Freivalds-style check
    against the oracle's definition on sampled entries."""
    M, N, K = 2088, 2048, 2048
    alpha, beta = 1.25, -0.75
    rng = _rng(77)
    A = _draw(rng, (K, M) if ta else (M, K), False)
    B = _draw(rng, (N, K) if tb else (K, N), False)
    C = _draw(rng, (M, N), False)
    dA, dB, dC = (torch.from_numpy(x).cuda() for x in (A, B, C))
    dg.dgemm_f64_ex(dA, dB, dC, alpha=alpha, beta=beta, transa=ta, transb=tb)
    got = dC.cpu().numpy()
    ii = rng.integers(0, M, size=400)
    jj = rng.integers(0, N, size=400)
    opA = A.T if ta else A
    opB = B.T if tb else B
    for i, j in zip(ii, jj):
        a_row = opA[i, :].copy().reshape(1, K)
        b_col = opB[:, j].copy().reshape(K, 1)
        want = np.array([[C[i, j]]])
        oracle.dgemm_oracle_general(False, False, alpha, a_row, b_col, beta, want)
        scale = abs(alpha) * (np.abs(a_row) @ np.abs(b_col)).item() + abs(beta) * abs(C[i, j])
        assert abs(got[i, j] - want[0, 0]) <= 2.0 * (K + 3) * U * scale
    # whole-matrix property: (alpha op(A) op(B) + beta C) x = alpha op(A) (op(B) x) + beta C x
    x = rng.integers(-2, 3, size=(N, 2)).astype(np.float64)
    lhs = got @ x
    rhs = alpha * (opA @ (opB @ x)) + beta * (C @ x)
    scale = abs(alpha) * (np.abs(opA) @ (np.abs(opB) @ np.abs(x))) + abs(beta) * (np.abs(C) @ np.abs(x))
    assert (np.abs(lhs - rhs) <= 4.0 * (K + N) * U * scale).all()


# One shape per kernel / tile configuration the library chooses by itself (checked with dgemm_plan),
# each with the scalars in the epilogue and, where K is split, in the partial-tile reduction.
CONFIG_SHAPES = [
    ((1536, 1408, 512), (dg.DGEMM_VARIANT_TMA_WS, 128, 128)),   # warp-specialised, 128-row tiles
    ((2048, 2304, 96), (dg.DGEMM_VARIANT_TMA_WS, 64, 128)),     # warp-specialised, 64-row tiles (K < 256)
    ((1040, 1000, 320), (dg.DGEMM_VARIANT_TMA_WS, 64, 128)),    # the same for a ragged M on a problem of moderate size
    ((700, 64, 520), (dg.DGEMM_VARIANT_TMA, 256, 32)),          # narrow tiles
    ((96, 1000, 300), (dg.DGEMM_VARIANT_TMA, 32, 128)),         # short tiles
    ((900, 146, 260), (dg.DGEMM_VARIANT_TMA, 128, 64)),         # half-width tiles
]


@pytest.mark.parametrize("shape,expect", CONFIG_SHAPES)
@pytest.mark.parametrize("alpha,beta", [(2.0, -3.0), (-1.0, 0.0)])
def test_scalars_in_every_tile_configuration(oracle, shape, expect, alpha, beta):
    M, N, K = shape
    pl = dg.dgemm_plan(M, N, K)
    assert (pl["variant"], pl["bm"], pl["bn"]) == expect, pl
    _case(oracle, M, N, K, False, False, alpha, beta, True, seed=sum(shape), pad=(2, 4, 7),
          c_fill=(np.nan if beta == 0.0 else None))
    _case(oracle, M, N, K, True, True, alpha, beta, False, seed=sum(shape) + 1)


@pytest.mark.parametrize("alpha,beta", [(2.0, -3.0), (-1.0, 0.0)])
def test_scalars_in_the_inline_kernel_with_64_row_tiles(oracle, alpha, beta):
    """The library's choice for a ragged M only on long problems (more than 256 k-blocks per resident
    CTA, too large for a full oracle comparison): forced here on a moderate one."""
    assert (dg.dgemm_plan(1600, 8192, 8192)["variant"], dg.dgemm_plan(1600, 8192, 8192)["bm"]) == (dg.DGEMM_VARIANT_TMA, 64)
    M, N, K = 1040, 1000, 320
    _case(oracle, M, N, K, False, False, alpha, beta, True, seed=77, pad=(2, 4, 7),
          c_fill=(np.nan if beta == 0.0 else None), variant=dg.DGEMM_VARIANT_TMA)
    _case(oracle, M, N, K, True, True, alpha, beta, False, seed=78, variant=dg.DGEMM_VARIANT_TMA)


def _runs_as_two_products(M, N, K):
    """The library's rule for running a ragged N as two products on a column split (the last two
    shapes below: there the transposed operands are rewritten first, as before)."""
    r = N % 128
    r32 = (r + 31) // 32 * 32
    wide = N >= 1024
    return N > 128 and 1 <= r <= (64 if wide else 32) and M * K * (128.0 - 1.2 * r32) > (2.0e8 if wide else 8.0e8)


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", [(2048, 2048, 512), (1024, 1024, 1024), (2088, 2048, 300), (600, 700, 500), (1000, 1537, 777),
                                   (2304, 2304, 64), (300, 260, 200), (1000, 1536, 256), (1010, 1536, 250),
                                   (3200, 400, 3000), (3000, 146, 3100),
                                   # a few tiles: K cut inside thread-block clusters
                                   (512, 512, 512), (320, 320, 320), (64, 64, 64), (200, 130, 96), (512, 512, 256),
                                   # narrow, short and half-width tiles
                                   (2000, 64, 1000), (1000, 32, 600), (3000, 90, 500), (32, 2000, 1000), (96, 1500, 700),
                                   (16, 640, 2048), (64, 64, 6000), (1000, 144, 512), (130, 70, 3000), (2048, 48, 2048)])
def test_transposed_operands_are_staged_without_a_pass(oracle, shape, integer):
    """op(A) = A^T, op(B) = B^T with operands the tensor-copy engine can address as they are stored
    (16-byte aligned, even leading dimension): the warp-specialised kernels and the inline kernel's
    tiles stage the transposed tiles themselves, so all four forms cost the launches of the
    untransposed product. Other kernels keep the transposing pass. Either way the result matches the
    oracle (M a multiple of 16 or not: one 3-D copy per stage of A^T, or box by box)."""
    M, N, K = shape
    counts = {}
    for ta, tb in FORMS:
        n0 = dg.dgemm_launch_count()
        _case(oracle, M, N, K, ta, tb, 1.0, 1.0, integer, seed=3000 + M + N + K, pad=(2, 4, 6))
        counts[(ta, tb)] = dg.dgemm_launch_count() - n0
    plan = dg.dgemm_plan(M, N, K, tma_addressable=False)  # (as planned without the bulk epilogue; the staging does not matter for the tile)
    plan = dg.dgemm_plan(M, N, K)
    tile = (plan["bm"], plan["bn"], plan["wtm"])
    native = ((plan["variant"] in (dg.DGEMM_VARIANT_TMA_WS, dg.DGEMM_VARIANT_TMA_CLUSTER) and plan["bn"] == 128 and plan["wtm"] == 64) or
              (plan["variant"] == dg.DGEMM_VARIANT_TMA and tile in ((64, 128, 64), (128, 64, 64), (256, 32, 64), (32, 128, 32)))) \
        and M % 2 == 0 and N % 2 == 0 and K % 2 == 0  # (even leading dimensions in every form with this padding)
    if _runs_as_two_products(M, N, K):  # both parts have to run on such kernels
        rest = dg.dgemm_plan(M, N % 128, K)
        native = native and rest["variant"] == dg.DGEMM_VARIANT_TMA and (rest["bm"], rest["bn"], rest["wtm"]) == (256, 32, 64)
    if native:
        assert len(set(counts.values())) == 1, (counts, plan)


def test_transposed_operand_that_cannot_be_used_in_place_takes_the_pass(oracle):
    """Odd leading dimension of the transposed operand, or an unaligned untransposed partner that is
    too small to repack: the transposing pass (and the generic staging) as before."""
    _case(oracle, 1024, 1024, 512, True, True, 1.0, 1.0, True, seed=77, pad=(3, 5, 7))
    _case(oracle, 300, 260, 200, False, True, 1.0, 1.0, True, seed=78, pad=(3, 4, 6))   # A odd, small: generic staging
    _case(oracle, 300, 260, 200, True, False, 2.0, -1.0, True, seed=79, pad=(2, 5, 6))  # B odd
    _case(oracle, 2048, 1024, 512, True, False, 1.0, 1.0, False, seed=80, pad=(2, 5, 6))  # B odd, large: packed, A^T native
