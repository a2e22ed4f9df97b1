"""Parity of the CUDA library (through the C ABI) against the CPU oracle. Needs a B200.

Bit-exact on integer-valued inputs. On uniform real inputs two bounds are asserted:
on the five benchmark configurations the stated criterion |dC_ij| <= 2*K*2^-53*(|A||B|)_ij, and
on every case the rigorous form 2*(K+1)*2^-53*(|C_in| + |A||B|)_ij (one more rounding against
C_in on each side), which is the only one that is a theorem for tiny K. Large cases use Freivalds'
check plus entries recomputed one by one by the oracle's triple loop. The largest error / bound
ratio per benchmark configuration is collected (see conftest.py: DGEMM_PARITY_REPORT).
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

from conftest import record_ratio

pytestmark = pytest.mark.gpu

GUARD = 64  # doubles of guard band on each side of every device buffer
GUARD_VALUE = -7.0e300


def _to_device(buf: torch.Tensor, offset_elems: int = 0):
    """Copy a padded host buffer into the middle of a larger device allocation with guard bands.
    Returns (whole allocation, 2-D view with the same shape/strides as the host buffer)."""
    rows, ld = buf.shape
    n = rows * ld
    whole = torch.full((n + 2 * GUARD + offset_elems,), GUARD_VALUE, dtype=torch.float64, device="cuda")
    start = GUARD + offset_elems
    whole[start:start + n] = buf.reshape(-1).cuda()
    view = whole[start:start + n].view(rows, ld)
    return whole, view


def _guards_intact(whole: torch.Tensor, n: int, offset_elems: int = 0) -> bool:
    start = GUARD + offset_elems
    return bool((whole[:start] == GUARD_VALUE).all() and (whole[start + n:] == GUARD_VALUE).all())


def run_gpu(prob: wl.Problem, variant=dg.DGEMM_VARIANT_AUTO, split_k=0, offset_elems=0):
    """Run dgemm_f64 on device copies of the problem; returns the resulting padded C buffer (host)."""
    dg.dgemm_set_variant(variant)
    dg.dgemm_set_split_k(split_k)
    try:
        wa, A = _to_device(prob.A_buf, offset_elems)
        wb, B = _to_device(prob.B_buf, offset_elems)
        wc, C = _to_device(prob.C_buf, offset_elems)
        before_a, before_b = wa.clone(), wb.clone()
        dg.dgemm_f64(A[:, :prob.K], B[:, :prob.N], C[:, :prob.N])
        assert dg.dgemm_last_device_status() == dg.DGEMM_OK
        out = C.cpu()
        assert _guards_intact(wc, prob.M * prob.ldc, offset_elems), "wrote outside the C buffer"
        # inputs untouched, bit for bit (NaN padding included)
        assert torch.equal(wa.view(torch.int64), before_a.view(torch.int64))
        assert torch.equal(wb.view(torch.int64), before_b.view(torch.int64))
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        dg.dgemm_set_split_k(0)
    assert wl.c_padding_intact(out, prob.N), "padding columns of C were modified"
    return out


def _check_full(oracle, prob: wl.Problem, out: torch.Tensor, stated: str = ""):
    """Element-by-element comparison with the oracle on the whole matrix. `stated`: name of a
    benchmark configuration; then the stated bound 2*K*u*(|A||B|)_ij is asserted as well and the
    largest error / bound ratio is recorded under that name."""
    want = prob.C.clone().contiguous().numpy()
    A = np.ascontiguousarray(prob.A.numpy())
    B = np.ascontiguousarray(prob.B.numpy())
    oracle.dgemm_oracle(A, B, want)
    got = out[:, :prob.N].numpy()
    if prob.integer:
        assert np.ascontiguousarray(got).tobytes() == want.tobytes(), "integer-valued inputs must match bit for bit"
        return 0.0
    # Stated bound 2*K*u*(|A||B|)_ij; when C_in != 0 each side rounds once more against |C_in|,
    # so the rigorous scale is (|C_in| + |A||B|)_ij with K+1 roundings.
    scale = oracle.abs_product(A, B, prob.C.numpy())
    bound = 2.0 * (prob.K + 1) * oracle.U * scale
    err = np.abs(got - want)
    assert np.isfinite(got).all()
    assert (err <= bound).all(), f"max err/bound = {(err / np.maximum(bound, 1e-300)).max()}"
    if stated:
        stated_bound = oracle.entry_bound(prob.K, oracle.abs_product(A, B))  # 2*K*u*(|A||B|)_ij: no C_in term
        ratio = float((err / np.maximum(stated_bound, 1e-300)).max())
        assert (err <= stated_bound).all(), f"stated bound: max err/bound = {ratio}"
        record_ratio(stated, ratio)
        return ratio
    return float((err / np.maximum(bound, 1e-300)).max())


# ---- config 1: 256^3, real then integer, C = 0 --------------------------------------------------

@pytest.mark.parametrize("integer", [False, True])
@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_AUTO, dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC,
                                     dg.DGEMM_VARIANT_NAIVE, dg.DGEMM_VARIANT_TMA_WS, dg.DGEMM_VARIANT_GENERIC_WS])
def test_config1(oracle, integer, variant):
    prob = wl.config1(integer)
    _check_full(oracle, prob, run_gpu(prob, variant), stated="config 1 (256^3)")


# ---- rungs of the ablation ladder: shared-memory tiles without a register tile, and the FMA
# ---- micro-kernel under the tensor-core kernels' staging, pipeline and epilogue --------------------

LADDER_VARIANTS = [dg.DGEMM_VARIANT_SMEM, dg.DGEMM_VARIANT_TMA_DFMA, dg.DGEMM_VARIANT_GENERIC_DFMA]


@pytest.mark.parametrize("integer", [False, True])
@pytest.mark.parametrize("variant", LADDER_VARIANTS)
def test_ladder_rungs_config1(oracle, integer, variant):
    prob = wl.config1(integer)
    _check_full(oracle, prob, run_gpu(prob, variant), stated="config 1 (256^3)")


@pytest.mark.parametrize("shape", [(1, 1, 1), (17, 13, 11), (127, 129, 47), (130, 260, 33), (257, 131, 100),
                                   (1000, 32, 600), (513, 33, 64), (1000, 1537, 777)])
@pytest.mark.parametrize("variant", LADDER_VARIANTS)
def test_ladder_rungs_ragged(oracle, shape, variant):
    """Ragged shapes with padded (even) leading dimensions, integer data (exact) and real data (bound)."""
    M, N, K = shape
    for integer in (True, False):
        prob = wl.make_problem(M, N, K, seed=400 + M + N + K, lda=K + 2 + (K & 1), ldb=N + 4 + (N & 1), ldc=N + 7,
                               integer=integer)
        _check_full(oracle, prob, run_gpu(prob, variant))


@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_TMA_DFMA, dg.DGEMM_VARIANT_GENERIC_DFMA])
def test_dfma_micro_kernel_split_k_and_odd_ld(oracle, variant):
    """The swapped micro-kernel shares split K, the stream-K tail and the epilogue forms with the tensor-core kernels."""
    prob = wl.make_problem(200, 150, 1000, seed=11, lda=1000, ldb=152, ldc=151, integer=True)
    _check_full(oracle, prob, run_gpu(prob, variant, split_k=7))
    prob = wl.make_problem(2304, 2304, 512, seed=12, integer=True)   # whole waves and a stream-K tail
    _check_full(oracle, prob, run_gpu(prob, variant))
    if variant == dg.DGEMM_VARIANT_GENERIC_DFMA:
        prob = wl.make_problem(300, 260, 200, seed=13, lda=203, ldb=265, ldc=267)
        _check_full(oracle, prob, run_gpu(prob, variant))


# ---- tiny and odd shapes, every variant, padded leading dimensions ---------------------------------

SMALL_SHAPES = [(1, 1, 1), (1, 7, 3), (5, 1, 2), (3, 3, 17), (17, 13, 11), (8, 8, 16), (16, 16, 15),
                (31, 33, 29), (64, 64, 64), (127, 129, 47), (128, 128, 16), (129, 127, 17), (130, 260, 33),
                (257, 131, 100), (200, 300, 1), (1000, 32, 600), (700, 20, 333), (513, 33, 64)]


@pytest.mark.parametrize("shape", SMALL_SHAPES)
@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC, dg.DGEMM_VARIANT_TMA_WS,
                                     dg.DGEMM_VARIANT_GENERIC_WS])
def test_small_shapes_integer_exact(oracle, shape, variant):
    M, N, K = shape
    # even leading dimensions so that both staging variants can run the same problem
    prob = wl.make_problem(M, N, K, seed=100 + M + N + K, lda=K + 2 + (K & 1), ldb=N + 4 + (N & 1),
                           ldc=N + 7, integer=True)
    _check_full(oracle, prob, run_gpu(prob, variant))


@pytest.mark.parametrize("shape", SMALL_SHAPES)
def test_small_shapes_real_odd_ld(oracle, shape):
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=200 + M + N + K, lda=K + 3, ldb=N + 5, ldc=N + 7)
    _check_full(oracle, prob, run_gpu(prob))


@pytest.mark.parametrize("offset", [1, 2, 3])
def test_unaligned_base_pointers(oracle, offset):
    """Base pointers that are only 8-byte aligned (odd element offset into the allocation)."""
    prob = wl.make_problem(150, 140, 70, seed=7, lda=72, ldb=144, ldc=141, integer=True)
    _check_full(oracle, prob, run_gpu(prob, offset_elems=offset))


# ---- split-K (partial tiles through the workspace, deterministic reduction) -------------------------

@pytest.mark.parametrize("split", [2, 3, 7, 64])
@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC, dg.DGEMM_VARIANT_TMA_WS,
                                     dg.DGEMM_VARIANT_GENERIC_WS])
def test_split_k(oracle, split, variant):
    prob = wl.make_problem(200, 150, 1000, seed=11, lda=1000, ldb=150 + 2, ldc=151, integer=True)
    _check_full(oracle, prob, run_gpu(prob, variant, split_k=split))
    prob = wl.make_problem(129, 257, 515, seed=12, lda=516, ldb=258, ldc=257)
    _check_full(oracle, prob, run_gpu(prob, variant, split_k=split))


def test_split_k_deterministic():
    prob = wl.make_problem(300, 200, 2048, seed=13)
    a = run_gpu(prob, split_k=8)
    b = run_gpu(prob, split_k=8)
    assert torch.equal(a.view(torch.int64), b.view(torch.int64))


# ---- config 2: square sweep ---------------------------------------------------------------------

CONFIG2_FULL_UP_TO = 2048  # the oracle recomputes the whole matrix up to here, samples beyond


@pytest.mark.parametrize("n", [n for n in wl.config2_sizes() if n <= CONFIG2_FULL_UP_TO])
def test_config2_full(oracle, n):
    prob = wl.config2(n)
    _check_full(oracle, prob, run_gpu(prob), stated="config 2 (sweep)")


def _check_sampled(oracle, prob: wl.Problem, out: torch.Tensor, nsamples: int, seed: int, stated: str = ""):
    ii, jj = wl.sample_indices(prob.M, prob.N, nsamples, seed)
    A, B, C0 = prob.A.numpy(), prob.B.numpy(), prob.C.numpy()
    want = oracle.dgemm_oracle_entries(A, B, C0, ii.numpy(), jj.numpy())
    got = out[:, :prob.N][ii, jj].numpy()
    if prob.integer:
        assert np.array_equal(got, want)
        return
    scale = oracle.dgemm_oracle_entries(A, B, C0, ii.numpy(), jj.numpy(), absolute=True)
    bound = 2.0 * (prob.K + 1) * oracle.U * scale
    err = np.abs(got - want)
    assert (err <= bound).all()
    if stated:
        stated_bound = oracle.entry_bound(prob.K, oracle.dgemm_oracle_entries(A, B, None, ii.numpy(), jj.numpy(), absolute=True))
        ratio = float((err / np.maximum(stated_bound, 1e-300)).max())
        assert (err <= stated_bound).all(), f"stated bound: max err/bound = {ratio}"
        record_ratio(stated, ratio)


def _check_freivalds(oracle, prob: wl.Problem, out: torch.Tensor, nvec: int = 20, seed: int = 99):
    X = oracle.freivalds_vectors(prob.N, nvec, seed)
    resid, tol = oracle.freivalds_residual(prob.A.numpy(), prob.B.numpy(), prob.C.numpy(),
                                           out[:, :prob.N].numpy(), X)
    if prob.integer:
        assert (resid == 0).all(), "integer-valued data: Freivalds' identity must hold exactly"
    else:
        assert (resid <= tol).all(), f"max resid/tol = {(resid / tol).max()}"


@pytest.mark.parametrize("n", [n for n in wl.config2_sizes() if n > CONFIG2_FULL_UP_TO])
def test_config2_large_sampled(oracle, n):
    prob = wl.config2(n)
    out = run_gpu(prob)
    _check_freivalds(oracle, prob, out)
    _check_sampled(oracle, prob, out, 2048, seed=n, stated="config 2 (sweep)")


# ---- config 3: 8192^3 -----------------------------------------------------------------------------

@pytest.mark.parametrize("integer", [False, True])
def test_config3_8192(oracle, integer):
    prob = wl.config3(integer=integer)
    out = run_gpu(prob)
    _check_freivalds(oracle, prob, out, nvec=20, seed=1)
    _check_sampled(oracle, prob, out, 4096, seed=1, stated="" if integer else "config 3 (8192^3)")


@pytest.mark.parametrize("flags", [4, 8, 12])
@pytest.mark.parametrize("n", [1024, 2304])
def test_tile_configurations(oracle, n, flags):
    """The other tile configurations (128-row CTA tiles, 32-row warp tiles) on square cases, one of
    them with a partial last wave."""
    prob = wl.make_problem(n, n, n, seed=n + 1, integer=True)
    dg.dgemm_set_test_flags(flags)
    try:
        out = run_gpu(prob)
    finally:
        dg.dgemm_set_test_flags(0)
    if n <= 1024:
        _check_full(oracle, prob, out)
    else:
        _check_freivalds(oracle, prob, out)
        _check_sampled(oracle, prob, out, 2048, seed=n)


# ---- config 4: ragged shapes, padded odd leading dimensions ---------------------------------------

@pytest.mark.parametrize("flags", [0, 16])
@pytest.mark.parametrize("idx", [0, 1, 2])
def test_config4_ragged(oracle, idx, flags):
    """flags 16: without the packing pass (the odd-leading-dimension case then uses generic staging)."""
    prob = wl.config4(idx)
    dg.dgemm_set_test_flags(flags)
    try:
        out = run_gpu(prob)
    finally:
        dg.dgemm_set_test_flags(0)
    _check_full(oracle, prob, out, stated="config 4 (%d,%d,%d)" % wl.CONFIG4_SHAPES[idx])


@pytest.mark.parametrize("offset", [0, 1])
def test_packing_pass_unaligned_operands(oracle, offset):
    """Odd leading dimensions and an odd element offset: A and B are packed into aligned scratch first
    (twice in a row: the second call reuses the scratch). Integer data, exact."""
    prob = wl.make_problem(700, 650, 1200, seed=61, lda=1203, ldb=655, ldc=657, integer=True)  # 1.1 GFLOP, 100 flop per packed byte: packed
    first = run_gpu(prob, offset_elems=offset)
    _check_full(oracle, prob, first)
    second = run_gpu(prob, offset_elems=offset)
    assert torch.equal(first.view(torch.int64), second.view(torch.int64))


@pytest.mark.parametrize("flags", [0, 4, 8, 12])
@pytest.mark.parametrize("idx", [0, 2])
def test_config4_ragged_integer(oracle, idx, flags):
    M, N, K = wl.CONFIG4_SHAPES[idx]
    prob = wl.make_problem(M, N, K, 2, lda=K + 3, ldb=N + 5, ldc=N + 7, integer=True)
    dg.dgemm_set_test_flags(flags)
    try:
        out = run_gpu(prob)
    finally:
        dg.dgemm_set_test_flags(0)
    _check_full(oracle, prob, out)


# ---- config 5: rank-k updates -------------------------------------------------------------------

@pytest.mark.parametrize("K", wl.CONFIG5_K)
def test_config5_rank_k(oracle, K):
    prob = wl.config5(K)
    out = run_gpu(prob)
    _check_freivalds(oracle, prob, out, nvec=20, seed=3)
    _check_sampled(oracle, prob, out, 4096, seed=3, stated="config 5 (16384^2 x %d)" % K)


# ---- degenerate cases and argument errors ------------------------------------------------------

def test_degenerate_and_errors():
    A = torch.zeros(4, 4, dtype=torch.float64, device="cuda")
    B = torch.zeros(4, 4, dtype=torch.float64, device="cuda")
    C0 = torch.tensor([[-0.0, float("nan")], [1.5, -2.0]], dtype=torch.float64, device="cuda")
    C = C0.clone()
    # K = 0: C untouched bit for bit
    assert dg.dgemm_f64_raw(2, 2, 0, A.data_ptr(), 1, B.data_ptr(), 2, C.data_ptr(), 2) == 0
    torch.cuda.synchronize()
    assert torch.equal(C.view(torch.int64), C0.view(torch.int64))
    # M = 0 / N = 0: no-op even with null pointers
    assert dg.dgemm_f64_raw(0, 5, 5, None, 5, None, 5, None, 5) == 0
    assert dg.dgemm_f64_raw(5, 0, 5, None, 5, None, 1, None, 1) == 0
    a, b, c = A.data_ptr(), B.data_ptr(), C.data_ptr()
    assert dg.dgemm_f64_raw(-1, 2, 2, a, 2, b, 2, c, 2, check=False) == -1
    assert dg.dgemm_f64_raw(2, 2, 2, a, 1, b, 2, c, 2, check=False) == -2
    assert dg.dgemm_f64_raw(2, 2, 2, a, 2, b, 1, c, 2, check=False) == -2
    assert dg.dgemm_f64_raw(2, 2, 2, a, 2, b, 2, c, 1, check=False) == -2
    assert dg.dgemm_f64_raw(2, 2, 2, None, 2, b, 2, c, 2, check=False) == -3
    assert dg.dgemm_f64_raw(2, 2, 2, a + 4, 2, b, 2, c, 2, check=False) == -4
    assert dg.dgemm_f64_raw(2, 2, 2, a, 2, b, 2, a + 8, 2, check=False) == -5
    with pytest.raises(dg.DgemmError):
        dg.dgemm_f64_raw(2, 2, 2, a, 2, b, 2, b, 2)
    # forced TMA variant on an odd leading dimension is refused, not silently rerouted
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA)
    try:
        big = torch.zeros(64, dtype=torch.float64, device="cuda")
        assert dg.dgemm_f64_raw(2, 2, 2, big.data_ptr(), 3, b, 2, c, 2, check=False) == -9
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    assert dg.dgemm_last_device_status() == 0


def test_nan_propagates_to_its_row_only():
    A = torch.ones(130, 40, dtype=torch.float64)
    A[77, 5] = float("nan")
    prob = wl.make_problem(130, 140, 40, seed=5)
    prob.A_buf.copy_(A)
    prob.B_buf.fill_(1.0)
    out = run_gpu(prob)
    assert torch.isnan(out[77]).all()
    assert torch.isfinite(torch.cat([out[:77], out[78:]])).all()


def test_all_ones_paper_driver():
    """The paper's driver (Section 2.1): A = B = C = 1 on 2048-sized operands gives 1 + K."""
    n = 2048
    A = torch.ones(n, n, dtype=torch.float64, device="cuda")
    B = torch.ones(n, n, dtype=torch.float64, device="cuda")
    C = torch.ones(n, n, dtype=torch.float64, device="cuda")
    dg.dgemm_f64(A, B, C)
    assert dg.dgemm_last_device_status() == 0
    assert bool((C == 2049.0).all())


def test_accumulates_into_c_and_k_split_calls(oracle):
    """Two successive calls over a K partition equal one call (exact on integer data)."""
    prob = wl.make_problem(140, 130, 96, seed=21, integer=True)
    one = run_gpu(prob)
    A, B, C = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    dg.dgemm_f64(A[:, :40], B[:40, :], C)
    dg.dgemm_f64(A[:, 40:], B[40:, :], C)
    torch.cuda.synchronize()
    assert torch.equal(C.cpu(), one)


@pytest.mark.parametrize("shape", [(300, 257, 129), (2500, 300, 200), (3072, 130, 64), (2300, 70, 2500), (3100, 33, 3073), (6200, 40, 2100),
                                   (6801, 40, 2100)])
def test_host_entry_point(oracle, shape):
    """Host buffers; the larger cases are streamed through the device in several blocks of rows
    (a ragged last block in the second case), the last three also with B in several panels of rows
    behind the first block, which is multiplied K panel by K panel (a ragged last panel, one row in the
    fifth case); in the last two cases three head blocks are multiplied against the arriving panels
    (their own C follows B and is added at the end) and the other four go through the ring of buffers,
    the last of them, in the last case, in two halves of 328 and 329 rows."""
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=31, lda=K + 3, ldb=N + 5, ldc=N + 7)
    want = prob.C.clone().contiguous().numpy()
    oracle.dgemm_oracle(np.ascontiguousarray(prob.A.numpy()), np.ascontiguousarray(prob.B.numpy()), want)
    scale = oracle.abs_product(prob.A.numpy(), prob.B.numpy(), prob.C.numpy())
    dg.dgemm_f64_host(prob.A, prob.B, prob.C)
    assert wl.c_padding_intact(prob.C_buf, prob.N)
    assert (np.abs(prob.C.numpy() - want) <= 2.0 * (prob.K + 1) * oracle.U * scale).all()


def test_non_default_stream(oracle):
    prob = wl.make_problem(256, 256, 512, seed=41, integer=True)
    A, B, C = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        dg.dgemm_f64(A, B, C, stream=s)
    assert dg.dgemm_last_device_status(s) == 0
    want = prob.C.clone().numpy()
    oracle.dgemm_oracle(prob.A.numpy(), prob.B.numpy(), want)
    assert np.array_equal(C.cpu().numpy(), want)


def test_bounded_wait_gives_up_and_reports(oracle):
    """A device-side wait that can never be satisfied ends after its limit with DGEMM_ERR_TIMEOUT in
    the status word; the context stays usable and the next GEMM is correct."""
    assert dg.dgemm_last_device_status() == 0
    assert dg.dgemm_selftest_wait_timeout(500) == 0
    assert dg.dgemm_last_device_status() == -8      # DGEMM_ERR_TIMEOUT, read and cleared
    assert dg.dgemm_last_device_status() == 0
    prob = wl.make_problem(200, 150, 90, seed=51, integer=True)
    _check_full(oracle, prob, run_gpu(prob))


SKINNY_SHAPES = [(32, 1000, 600), (16, 513, 129), (96, 500, 300), (160, 384, 512), (20, 129, 77), (417, 260, 200),
                 (1000, 48, 600), (1000, 96, 333), (513, 80, 64), (2000, 64, 2048), (300, 97, 128),
                 (1000, 146, 300), (700, 130, 520), (257, 416, 100), (129, 190, 64)]


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", SKINNY_SHAPES)
def test_skinny_shapes_auto(oracle, shape, integer):
    """Shapes that the library's own choice sends to the 32 x 128 tile (short M), to one to three
    columns of 256 x 32 tiles (N <= 96) and to 128 x 64 tiles (N just above a multiple of 128), with
    aligned operands (TMA staging) and a padded C."""
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=300 + M + N + K, lda=K + 2 + (K & 1), ldb=N + 4 + (N & 1), ldc=N + 7,
                           integer=integer)
    _check_full(oracle, prob, run_gpu(prob))


@pytest.mark.parametrize("n", [200, 1024])
def test_a_and_b_may_be_the_same_buffer(oracle, n):
    """A and B are read only and may alias each other (C += A A); C overlapping either is refused."""
    rng = np.random.Generator(np.random.PCG64(n))
    A = rng.integers(-4, 5, (n, n)).astype(np.float64)
    C = rng.integers(-4, 5, (n, n)).astype(np.float64)
    dA, dC = torch.from_numpy(A).cuda(), torch.from_numpy(C).cuda()
    dg.dgemm_f64(dA, dA, dC)
    assert dg.dgemm_last_device_status() == dg.DGEMM_OK
    want = C.copy()
    oracle.dgemm_oracle(A, A.copy(), want)
    assert np.array_equal(dC.cpu().numpy(), want)
    assert dg.dgemm_f64(dA, dA, dA, check=False) == dg.binding.DGEMM_ERR_ALIAS
    assert dg.dgemm_f64_ex(dA, dC, dC, alpha=1.0, beta=0.0, check=False) == dg.binding.DGEMM_ERR_ALIAS


@pytest.mark.parametrize("shape", [(1024, 1024, 1024), (2088, 2048, 2048), (300, 200, 100), (4097, 31, 4099)])
def test_calls_can_be_captured_into_a_cuda_graph(shape):
    """After a first call outside capture (allocations, kernel attributes), dgemm_f64 calls recorded
    in a CUDA graph replay correctly, programmatic launches and reduction kernels included."""
    M, N, K = shape
    g0 = torch.Generator(device="cuda").manual_seed(M)
    A = torch.randint(-3, 4, (M, K), device="cuda", generator=g0).double()
    B = torch.randint(-3, 4, (K, N), device="cuda", generator=g0).double()
    C = torch.zeros(M, N, dtype=torch.float64, device="cuda")
    dg.dgemm_f64(A, B, C)
    torch.cuda.synchronize()
    once = C.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        dg.dgemm_f64(A, B, C)
        dg.dgemm_f64(A, B, C)
    C.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert dg.dgemm_last_device_status() == dg.DGEMM_OK
    assert torch.equal(C, 4 * once)  # exact: small integers


def test_release_scratch_and_carry_on(oracle):
    """The workspace, the packing scratch and the host entry point's pool can be given back at any
    quiet moment; the next calls allocate them again and give the same results."""
    prob = wl.make_problem(700, 520, 300, seed=71, lda=303, ldb=525, ldc=527, integer=True)   # generic staging, K split
    big = wl.make_problem(700, 650, 1200, seed=72, lda=1203, ldb=655, ldc=657, integer=True)  # packing pass
    first = [run_gpu(prob), run_gpu(big)]
    hostp = wl.make_problem(2500, 300, 200, seed=73, integer=True)
    want = hostp.C.clone().contiguous().numpy()
    oracle.dgemm_oracle(np.ascontiguousarray(hostp.A.numpy()), np.ascontiguousarray(hostp.B.numpy()), want)
    c0 = hostp.C.clone()
    dg.dgemm_f64_host(hostp.A, hostp.B, hostp.C)
    assert np.array_equal(hostp.C.numpy(), want)
    assert dg.dgemm_release_scratch() == dg.DGEMM_OK
    assert dg.dgemm_release_scratch() == dg.DGEMM_OK   # nothing left to free: still fine
    second = [run_gpu(prob), run_gpu(big)]
    for a, b in zip(first, second):
        assert torch.equal(a.view(torch.int64), b.view(torch.int64))
    _check_full(oracle, prob, second[0])
    hostp.C.copy_(c0)
    dg.dgemm_f64_host(hostp.A, hostp.B, hostp.C)
    assert np.array_equal(hostp.C.numpy(), want)


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", [(2000, 1064, 2000), (2100, 1300, 2050), (3000, 146, 3100), (3200, 400, 3000)])
def test_ragged_n_on_a_large_problem_runs_as_two_products(oracle, shape, integer):
    """N just above a multiple of 128 on a large problem: the full tile columns and the narrow
    remainder are separate launches on disjoint columns of C (padded, odd ldc in the second case:
    both parts go through the staged epilogue). The last two are tall problems of one and three
    tile columns plus a remainder of less than 32 columns."""
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=81, ldc=N + (7 if N == 1300 else 0), integer=integer)
    n0 = dg.dgemm_launch_count()
    out = run_gpu(prob)
    assert dg.dgemm_launch_count() - n0 >= 2
    _check_freivalds(oracle, prob, out)
    _check_sampled(oracle, prob, out, 4096, seed=5)
    # the columns on both sides of the cut, every row
    import numpy as _np
    cut = N - N % 128
    ii = _np.repeat(_np.arange(M), 4)
    jj = _np.tile(_np.array([cut - 1, cut, cut + 1, N - 1]), M)
    want = oracle.dgemm_oracle_entries(prob.A.numpy(), prob.B.numpy(), prob.C.numpy(), ii, jj)
    got = out[:, :N].numpy()[ii, jj]
    if integer:
        assert _np.array_equal(got, want)
    else:
        scale = oracle.dgemm_oracle_entries(prob.A.numpy(), prob.B.numpy(), prob.C.numpy(), ii, jj, absolute=True)
        assert (_np.abs(got - want) <= 2.0 * (K + 1) * oracle.U * scale).all()
