"""Extreme aspect ratios (very tall, very wide, very deep, single rows and columns) for dgemm_f64
and sgemm_f32: sampled entries against the oracle's definition, bit for bit on integer data, plus
row and column sums over the whole result. Needs a B200."""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg

pytestmark = pytest.mark.gpu

SHAPES = [(600000, 40, 24, (0, 0, 0)), (600001, 33, 17, (1, 1, 1)), (24, 600000, 40, (0, 0, 0)),
          (17, 600001, 33, (1, 1, 1)), (64, 64, 300000, (0, 0, 0)), (1, 1, 1, (0, 0, 0)), (1, 100000, 1, (0, 0, 0)),
          (100000, 1, 1, (0, 0, 0)), (2, 3, 100001, (1, 0, 0)), (70000, 70, 70, (0, 0, 0)), (4097, 4099, 129, (3, 1, 1))]


@pytest.mark.parametrize("single", [False, True])
@pytest.mark.parametrize("M,N,K,pad", SHAPES)
def test_extreme_shapes(oracle, M, N, K, pad, single):
    rng = np.random.Generator(np.random.PCG64(M + N + K))
    ntype, ttype = (np.float32, torch.float32) if single else (np.float64, torch.float64)
    A = rng.integers(-3, 4, (M, K)).astype(ntype)
    B = rng.integers(-3, 4, (K, N)).astype(ntype)
    C = rng.integers(-3, 4, (M, N)).astype(ntype)

    def dev(x, p):
        buf = torch.full((x.shape[0], x.shape[1] + p), float("nan"), dtype=ttype, device="cuda")
        buf[:, :x.shape[1]] = torch.from_numpy(x).cuda()
        return buf, buf[:, :x.shape[1]]

    (_, dA), (_, dB), (bufC, dC) = dev(A, pad[0]), dev(B, pad[1]), dev(C, pad[2])
    if single:
        dg.sgemm_f32(dA, dB, dC)
        assert dg.sgemm_last_device_status() == dg.DGEMM_OK
    else:
        dg.dgemm_f64(dA, dB, dC)
        assert dg.dgemm_last_device_status() == dg.DGEMM_OK
    got = dC.cpu().numpy()
    if pad[2]:
        assert bool(torch.isnan(bufC[:, N:]).all())
    n = min(3000, M * N)
    ii, jj = rng.integers(0, M, n), rng.integers(0, N, n)
    entries = oracle.sgemm_oracle_entries if single else oracle.dgemm_oracle_entries
    want = entries(A, B, C, ii, jj)
    assert np.array_equal(got[ii, jj], want)
    # every entry takes part in a row sum and a column sum (exact: small integers)
    a64, b64, c64, g64 = (x.astype(np.float64) for x in (A, B, C, got))
    assert np.array_equal(g64.sum(axis=1), c64.sum(axis=1) + a64 @ b64.sum(axis=1))
    assert np.array_equal(g64.sum(axis=0), c64.sum(axis=0) + a64.sum(axis=0) @ b64)


@pytest.mark.parametrize("single", [False, True])
def test_subnormal_values_are_not_flushed(oracle, single):
    """B holds small integer multiples of the smallest subnormal, A small integers: every product and
    partial sum is an exactly representable subnormal, so the result must equal the oracle's bit
    for bit; any flush-to-zero on the way would show."""
    ntype, ttype = (np.float32, torch.float32) if single else (np.float64, torch.float64)
    tiny = np.finfo(ntype).smallest_subnormal
    rng = np.random.Generator(np.random.PCG64(9))
    M, N, K = 200, 150, 96
    A = rng.integers(-3, 4, (M, K)).astype(ntype)
    B = (rng.integers(-3, 4, (K, N)).astype(ntype) * tiny).astype(ntype)
    C = (rng.integers(-3, 4, (M, N)).astype(ntype) * tiny).astype(ntype)
    assert np.count_nonzero(B) > 0 and np.abs(B).max() < np.finfo(ntype).tiny
    dA, dB, dC = (torch.from_numpy(x).cuda() for x in (A, B, C))
    want = C.copy()
    if single:
        dg.sgemm_f32(dA, dB, dC)
        oracle.sgemm_oracle(A, B, want)
    else:
        dg.dgemm_f64(dA, dB, dC)
        oracle.dgemm_oracle(A, B, want)
    got = dC.cpu().numpy()
    assert np.count_nonzero(want) > 0
    assert got.tobytes() == want.tobytes()
