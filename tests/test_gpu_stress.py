"""Repeated-run stress test of the stage hand-over in the pipelined kernels. Needs a B200.

A stage of the operand pipeline must not be refilled while a warp's fragment loads from it are
still outstanding. When that was violated, one warp's 8-row blocks of a tile came out wrong in a
fraction of the runs, mostly early in the kernel, on rank-k shapes whose tiles are short (K = 64),
and reliably so with the optional accelerations switched off (slower epilogues, more copies per
stage). The test repeats exactly that: integer-valued data (every correct result is bit-identical
to the oracle's), many runs, the settings of the test flags (including the 128-row tile), all staging variants.
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rank_k_case(oracle):
    prob = wl.make_problem(8192, 8192, 64, seed=3, integer=True)
    want = prob.C.clone().numpy()
    oracle.dgemm_oracle(prob.A.numpy(), prob.B.numpy(), want)
    return prob, torch.from_numpy(want)


@pytest.mark.parametrize("flags", [3, 1, 2, 0, 7, 4, 8, 12, 15, 32])
@pytest.mark.parametrize("variant", [dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC, dg.DGEMM_VARIANT_TMA_WS,
                                     dg.DGEMM_VARIANT_GENERIC_WS])
def test_rank_k_repeated_runs_bit_exact(rank_k_case, flags, variant):
    prob, want = rank_k_case
    A, B, C0 = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    want_dev = want.cuda()
    # a small call first: it takes the stream-K path and allocates the workspace, which is the
    # situation in which the failure was most frequent
    a = torch.ones(256, 256, dtype=torch.float64, device="cuda")
    c = torch.zeros(256, 256, dtype=torch.float64, device="cuda")
    dg.dgemm_f64(a, a, c)
    dg.dgemm_set_test_flags(flags)
    dg.dgemm_set_variant(variant)
    try:
        reps = 12 if variant in (dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_TMA_WS) else 4
        for rep in range(reps):
            C = C0.clone()
            dg.dgemm_f64(A, B, C)
            assert dg.dgemm_last_device_status() == 0
            wrong = int((C != want_dev).sum())
            assert wrong == 0, f"run {rep}: {wrong} wrong entries (flags {flags}, variant {variant})"
    finally:
        dg.dgemm_set_test_flags(0)
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    assert bool((c == 256.0).all())


@pytest.mark.parametrize("n", [2304, 2560, 3072])
@pytest.mark.parametrize("kernel", ["auto", "inline", "ws_two_ctas"])
def test_square_repeated_runs_bit_exact(oracle, n, kernel):
    """Sizes with a partial last wave (stream-K tail), repeated; exact against the oracle's entries
    on sampled positions and against the first run everywhere. `auto` is the warp-specialised
    kernel with 128-row tiles at these sizes; the other two are its 64-row form and the inline kernel."""
    if kernel == "inline":
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA)
    elif kernel == "ws_two_ctas":
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA_WS)
        dg.dgemm_set_test_flags(32)
    try:
        _square_repeated(oracle, n)
    finally:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        dg.dgemm_set_test_flags(0)


def _square_repeated(oracle, n):
    prob = wl.make_problem(n, n, n, seed=n, integer=True)
    A, B, C0 = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    ii, jj = wl.sample_indices(n, n, 4096, seed=n)
    want = oracle.dgemm_oracle_entries(prob.A.numpy(), prob.B.numpy(), prob.C.numpy(), ii.numpy(), jj.numpy())
    first = None
    for rep in range(6):
        C = C0.clone()
        dg.dgemm_f64(A, B, C)
        assert dg.dgemm_last_device_status() == 0
        got = C[ii.cuda(), jj.cuda()].cpu().numpy()
        assert np.array_equal(got, want)
        if first is None:
            first = C
        else:
            assert torch.equal(first, C), f"run {rep} differs from run 0"


@pytest.mark.parametrize("flags", [0, 2])
@pytest.mark.parametrize("split", [1, 2, 8])
def test_cluster_kernel_repeated_runs_bit_exact(oracle, flags, split):
    """The cluster split-K kernel with long K runs per CTA (every stage refilled many times, which
    the library's own choice never asks of it) and more clusters than are resident at once."""
    M, N, K = 1000, 1100, 1000
    prob = wl.make_problem(M, N, K, seed=11, integer=True)
    want = prob.C.clone().numpy()
    oracle.dgemm_oracle(prob.A.numpy(), prob.B.numpy(), want)
    want_dev = torch.from_numpy(want).cuda()
    A, B, C0 = prob.A.cuda(), prob.B.cuda(), prob.C.cuda()
    dg.dgemm_set_test_flags(flags)
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA_CLUSTER)
    dg.dgemm_set_split_k(split)
    try:
        for rep in range(10):
            C = C0.clone()
            dg.dgemm_f64(A, B, C)
            assert dg.dgemm_last_device_status() == 0
            wrong = int((C != want_dev).sum())
            assert wrong == 0, f"run {rep}: {wrong} wrong entries (flags {flags}, clusters of {split})"
    finally:
        dg.dgemm_set_test_flags(0)
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        dg.dgemm_set_split_k(0)
