"""The allocation-free entry point ``dgemm_f64_static_ws`` against ``dgemm_f64``. Needs a B200.

``dgemm_f64_static_ws`` exists for callers that must not allocate device memory at the time of
the call (a lock shared with an allocator, a fixed memory budget, a latency-critical loop): its
split-K partial tiles live in a fixed device array inside the library. The test calls it through
the C ABI twice in a row (the second call finds the first call's leftovers in the array) and
compares each result with the regular entry point's on the same inputs, within the bound the
other parity tests use (bit for bit on integer-valued data). It also checks the capacity limit
and that the free device memory does not shrink across the calls.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

pytestmark = pytest.mark.gpu

U = 2.0 ** -53


def _device_copies(prob):
    return prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()


def _bound(prob):
    """2*(K+1)*2^-53*(|C_in| + |A||B|)_ij, evaluated on the device in float64."""
    A, B, C = prob.A.cuda().abs(), prob.B.cuda().abs(), prob.C.cuda().abs()
    return (2.0 * (prob.K + 1) * U * (C + A @ B)).cpu().numpy()


@pytest.mark.parametrize("shape,ld,integer,split", [
    ((300, 260, 1000), (1000, 260, 260), True, 0),     # 9 tiles, library-chosen split, TMA staging
    ((300, 260, 1000), (1003, 265, 267), False, 0),    # odd leading dimensions: generic staging
    ((129, 257, 515), (516, 258, 257), False, 7),      # forced split with a ragged last partition
    ((1000, 1000, 333), (334, 1000, 1001), True, 2),   # 64 tiles x 2 = the full capacity
])
def test_static_ws_matches_regular_entry_point(shape, ld, integer, split):
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=77, lda=ld[0], ldb=ld[1], ldc=ld[2], integer=integer)
    A, B, C_ref = _device_copies(prob)
    dg.dgemm_f64(A[:, :K], B[:, :N], C_ref[:, :N])
    assert dg.dgemm_last_device_status() == 0
    ref = C_ref.cpu()
    bound = None if integer else _bound(prob)

    # first call also does the per-device set-up; measure free memory around the later calls
    _, _, C0 = _device_copies(prob)
    dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], C0[:, :N], split_k=split)
    torch.cuda.synchronize()
    outs = [C0.cpu()]
    C1, C2 = prob.C_buf.cuda(), prob.C_buf.cuda()
    free_before, _ = torch.cuda.mem_get_info()
    for Cx in (C1, C2):  # two calls in a row, sharing the array
        dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], Cx[:, :N], split_k=split)
    assert dg.dgemm_last_device_status() == 0
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after >= free_before, "the entry point must not allocate device memory"
    outs += [C1.cpu(), C2.cpu()]

    for out in outs:
        assert wl.c_padding_intact(out, N)
        got, want = out[:, :N].numpy(), ref[:, :N].numpy()
        if integer:
            assert np.ascontiguousarray(got).tobytes() == np.ascontiguousarray(want).tobytes()
        else:
            assert (np.abs(got - want) <= bound).all()
    # same inputs, same split: the repeated calls agree bit for bit (fixed reduction order)
    assert torch.equal(outs[1].view(torch.int64), outs[2].view(torch.int64))


def test_static_ws_capacity_and_arguments():
    n = 1536  # 12 x 12 = 144 tiles: beyond the 128-tile array whatever the split
    A = torch.zeros(n, n, dtype=torch.float64, device="cuda")
    B = torch.zeros(n, n, dtype=torch.float64, device="cuda")
    C = torch.ones(n, n, dtype=torch.float64, device="cuda")
    assert dg.dgemm_f64_static_ws(A, B, C, check=False) == -10
    with pytest.raises(dg.DgemmError):
        dg.dgemm_f64_static_ws(A, B, C, split_k=2)
    # 64 tiles fit with split 2 but not with split 3
    m = 1024
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=3, check=False) == -10
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=-1, check=False) == -9
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=2) == 0
    # K <= 16: a single k-block, runs unsplit; M = 0: nothing to do
    assert dg.dgemm_f64_static_ws(A[:m, :8], B[:8, :m], C[:m, :m]) == 0
    assert dg.dgemm_f64_static_ws(A[:0, :m], B[:m, :m], C[:0, :m]) == 0
    assert dg.dgemm_last_device_status() == 0
    assert bool((C == 1.0).all())  # zero operands: C unchanged everywhere, refused calls included
