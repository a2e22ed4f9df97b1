"""The allocation-free entry point ``dgemm_f64_static_ws`` against the CPU oracle and ``dgemm_f64``.
Needs a B200.

``dgemm_f64_static_ws`` exists for callers that must not allocate device memory at the time of
the call (a lock shared with an allocator, a fixed memory budget, a latency-critical loop): its
split-K partial tiles live in a fixed device array inside the library. The tests call it through
the C ABI several times in a row. Between the checked calls the array is deliberately filled with
the partial tiles of another product (A scaled by -3) over the same tiles and partitions, so a
slot that is read without having been rewritten shows up as a wrong result. Every result is
compared element by element with the oracle (bit for bit on integer-valued data, within the
bound of the other parity tests on real data) and with the regular entry point. The tests also
check the capacity rules and that the free device memory does not shrink across the calls.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _device_copies(prob):
    return prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()


def _oracle_result(oracle, prob):
    """(expected C, rigorous bound 2*(K+1)*2^-53*(|C_in| + |A||B|)_ij) from the oracle alone."""
    A = np.ascontiguousarray(prob.A.numpy())
    B = np.ascontiguousarray(prob.B.numpy())
    want = prob.C.clone().contiguous().numpy()
    oracle.dgemm_oracle(A, B, want)
    bound = None if prob.integer else 2.0 * (prob.K + 1) * oracle.U * oracle.abs_product(A, B, prob.C.numpy())
    return want, bound


def _assert_matches(out, want, bound, N, integer):
    assert wl.c_padding_intact(out, N)
    got = out[:, :N].numpy()
    if integer:
        assert np.ascontiguousarray(got).tobytes() == np.ascontiguousarray(want).tobytes()
    else:
        assert np.isfinite(got).all()
        assert (np.abs(got - want) <= bound).all()


CASES = [
    ((300, 260, 1000), (1000, 260, 260), True, 0),     # 9 tiles, library-chosen split, TMA staging
    ((300, 260, 1000), (1003, 265, 267), False, 0),    # odd leading dimensions: generic staging
    ((129, 257, 515), (516, 258, 257), False, 7),      # forced split with a ragged last partition
    ((1000, 1000, 333), (334, 1000, 1001), True, 2),   # 64 tiles x 2 = the full capacity
]


@pytest.mark.parametrize("shape,ld,integer,split", CASES)
def test_static_ws_matches_oracle_and_regular_entry_point(oracle, shape, ld, integer, split):
    M, N, K = shape
    prob = wl.make_problem(M, N, K, seed=77, lda=ld[0], ldb=ld[1], ldc=ld[2], integer=integer)
    want, bound = _oracle_result(oracle, prob)
    A, B, C_ref = _device_copies(prob)
    dg.dgemm_f64(A[:, :K], B[:, :N], C_ref[:, :N])
    assert dg.dgemm_last_device_status() == 0
    _assert_matches(C_ref.cpu(), want, bound, N, integer)   # the regular entry point, for reference

    # another product over the same tiles and partitions, to leave wrong partial tiles behind
    A_other = A.clone()
    A_other[:, :K] *= -3.0

    def spoil_array():
        scratch_c = prob.C_buf.cuda()
        dg.dgemm_f64_static_ws(A_other[:, :K], B[:, :N], scratch_c[:, :N], split_k=split)

    # first call also does the per-device set-up; measure free memory around the later calls
    _, _, C0 = _device_copies(prob)
    dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], C0[:, :N], split_k=split)
    torch.cuda.synchronize()
    outs = [C0.cpu()]
    C1, C2 = prob.C_buf.cuda(), prob.C_buf.cuda()
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], C1[:, :N], split_k=split)   # two calls in a row ...
    dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], C2[:, :N], split_k=split)   # ... sharing the array
    assert dg.dgemm_last_device_status() == 0
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after >= free_before, "the entry point must not allocate device memory"
    outs += [C1.cpu(), C2.cpu()]
    spoil_array()
    C3 = prob.C_buf.cuda()
    dg.dgemm_f64_static_ws(A[:, :K], B[:, :N], C3[:, :N], split_k=split)   # finds the other product's leftovers
    assert dg.dgemm_last_device_status() == 0
    outs.append(C3.cpu())

    for out in outs:
        _assert_matches(out, want, bound, N, integer)
    # same inputs, same split: repeated calls agree bit for bit (fixed reduction order), whatever the array held
    for out in outs[1:]:
        assert torch.equal(outs[0].view(torch.int64), out.view(torch.int64))


def test_static_ws_two_calls_on_a_side_stream(oracle):
    """Two calls back to back on one non-default stream (stream order serialises them), the array
    holding another product's partial tiles beforehand."""
    prob = wl.make_problem(260, 300, 777, seed=78, lda=778, ldb=300, ldc=303, integer=True)
    want, _ = _oracle_result(oracle, prob)
    A, B, _ = _device_copies(prob)
    A_other = A.clone()
    A_other[:, :prob.K] *= -3.0
    Cs = [prob.C_buf.cuda() for _ in range(3)]
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        dg.dgemm_f64_static_ws(A_other[:, :prob.K], B[:, :prob.N], Cs[0][:, :prob.N], split_k=5, stream=s)
        dg.dgemm_f64_static_ws(A[:, :prob.K], B[:, :prob.N], Cs[1][:, :prob.N], split_k=5, stream=s)
        dg.dgemm_f64_static_ws(A[:, :prob.K], B[:, :prob.N], Cs[2][:, :prob.N], split_k=5, stream=s)
    assert dg.dgemm_last_device_status(s) == 0
    for C in Cs[1:]:
        _assert_matches(C.cpu(), want, None, prob.N, True)


def test_static_ws_capacity_and_arguments(oracle):
    n = 1536  # 12 x 12 = 144 tiles: beyond the 128-tile array for any split >= 1... but only a split uses it
    A = torch.zeros(n, n, dtype=torch.float64, device="cuda")
    B = torch.zeros(n, n, dtype=torch.float64, device="cuda")
    C = torch.ones(n, n, dtype=torch.float64, device="cuda")
    assert dg.dgemm_f64_static_ws(A, B, C, split_k=2, check=False) == -10
    with pytest.raises(dg.DgemmError):
        dg.dgemm_f64_static_ws(A, B, C, split_k=3)
    # one partition needs no array: explicit, chosen by the library for a large problem, or K <= 16
    assert dg.dgemm_f64_static_ws(A, B, C, split_k=1) == 0
    assert dg.dgemm_f64_static_ws(A, B, C) == 0
    assert dg.dgemm_f64_static_ws(A[:, :8], B[:8, :], C, split_k=4) == 0
    # 64 tiles fit with split 2 but not with split 3
    m = 1024
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=3, check=False) == -10
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=-1, check=False) == -9
    assert dg.dgemm_f64_static_ws(A[:m, :m], B[:m, :m], C[:m, :m], split_k=2) == 0
    # M = 0: nothing to do
    assert dg.dgemm_f64_static_ws(A[:0, :m], B[:m, :m], C[:0, :m]) == 0
    assert dg.dgemm_last_device_status() == 0
    assert bool((C == 1.0).all())  # zero operands: C unchanged everywhere, refused calls included

    # 72 tiles with the library's choice: two partitions would need 144 slots, so it runs unsplit
    prob = wl.make_problem(1024, 1152, 200, seed=79, integer=True)
    want, _ = _oracle_result(oracle, prob)
    dA, dB, dC = _device_copies(prob)
    assert dg.dgemm_f64_static_ws(dA, dB, dC) == 0
    assert dg.dgemm_last_device_status() == 0
    _assert_matches(dC.cpu(), want, None, prob.N, True)
