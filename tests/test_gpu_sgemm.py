"""Parity of the single-precision entry point ``sgemm_f32`` against the binary32 CPU oracle.
Needs a B200.

Bit-exact on integer-valued inputs; |dC_ij| <= 2 K 2^-24 (|C| + |A||B|)_ij on uniform real inputs
(each side errs by at most (K+1) u32 times that scale from the exact value; K+1 <= 2K for K >= 1).
"""
import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg

pytestmark = pytest.mark.gpu

U32 = 2.0 ** -24


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _draw(rng, shape, integer):
    if integer:
        return rng.integers(-4, 5, size=shape).astype(np.float32)
    return rng.uniform(-1.0, 1.0, size=shape).astype(np.float32)


def _padded_dev(x, ld, offset=0):
    rows, cols = x.shape
    whole = torch.full((rows * ld + offset + 8,), float("nan"), dtype=torch.float32, device="cuda")
    buf = whole[offset:offset + rows * ld].view(rows, ld)
    buf[:, :cols] = torch.from_numpy(x).cuda()
    return buf, buf[:, :cols]


def _run(M, N, K, integer, seed, pad=(0, 0, 0), offset=0):
    rng = _rng(seed)
    A, B, C = _draw(rng, (M, K), integer), _draw(rng, (K, N), integer), _draw(rng, (M, N), integer)
    bufA, dA = _padded_dev(A, K + pad[0], offset)
    bufB, dB = _padded_dev(B, N + pad[1], offset)
    bufC, dC = _padded_dev(C, N + pad[2], 0)
    a0, b0 = bufA.clone(), bufB.clone()
    dg.sgemm_f32(dA, dB, dC)
    assert dg.sgemm_last_device_status() == dg.DGEMM_OK
    assert bool(torch.isnan(bufC[:, N:]).all()), "padding columns of C were modified"
    assert torch.equal(a0.view(torch.int32), bufA.view(torch.int32)) and torch.equal(b0.view(torch.int32), bufB.view(torch.int32))
    return A, B, C, dC.cpu().numpy()


def _check(oracle, A, B, C, got, integer):
    want = C.copy()
    oracle.sgemm_oracle(A, B, want)
    if integer:
        assert np.ascontiguousarray(got).tobytes() == want.tobytes()
        return
    K = A.shape[1]
    scale = np.abs(C).astype(np.float64) + np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64)
    err = np.abs(got.astype(np.float64) - want.astype(np.float64))
    bound = 2.0 * K * U32 * scale
    assert np.isfinite(got).all()
    assert (err <= bound).all(), f"max err/bound = {(err / np.maximum(bound, 1e-300)).max()}"


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape", [(256, 256, 256), (128, 128, 32), (1, 1, 1), (3, 5, 7), (129, 127, 33), (333, 257, 190),
                                   (1000, 96, 600), (64, 1000, 45), (513, 33, 64), (700, 20, 333),
                                   # short M (64-row tiles), narrow N (64-column tiles), both, and the last wave cut in K
                                   (32, 2000, 1000), (150, 700, 1200), (190, 260, 515), (2000, 64, 1000), (3000, 40, 700),
                                   (1500, 160, 900), (1000, 190, 333), (60, 50, 4000), (40, 192, 2048), (9000, 32, 256)])
def test_small_shapes_dense(oracle, shape, integer):
    A, B, C, got = _run(*shape, integer, seed=sum(shape))
    _check(oracle, A, B, C, got, integer)


@pytest.mark.parametrize("integer", [True, False])
@pytest.mark.parametrize("shape,pad,offset", [((333, 257, 190), (3, 5, 7), 0), ((200, 130, 77), (1, 2, 0), 1),
                                              ((1000, 1537, 777), (3, 5, 7), 0), ((260, 256, 64), (4, 8, 4), 2),
                                              ((384, 160, 96), (0, 0, 1), 3)])
def test_padded_and_unaligned(oracle, shape, pad, offset, integer):
    """Odd leading dimensions and bases off the 16-byte boundary (packing pass), padded C."""
    A, B, C, got = _run(*shape, integer, seed=11 + offset, pad=pad, offset=offset)
    _check(oracle, A, B, C, got, integer)


def test_k_zero_and_empty():
    C = torch.ones(5, 7, dtype=torch.float32, device="cuda")
    dg.sgemm_f32(torch.zeros(5, 0, dtype=torch.float32, device="cuda"), torch.zeros(0, 7, dtype=torch.float32, device="cuda"), C)
    assert bool((C == 1).all())
    dg.sgemm_f32(torch.zeros(0, 4, dtype=torch.float32, device="cuda"), torch.zeros(4, 7, dtype=torch.float32, device="cuda"),
                 torch.zeros(0, 7, dtype=torch.float32, device="cuda"))


def test_all_ones_driver():
    """The paper's driver: every matrix is all ones; each entry becomes 1 + K."""
    M, N, K = 2088, 2048, 2048
    A = torch.ones(M, K, dtype=torch.float32, device="cuda")
    B = torch.ones(K, N, dtype=torch.float32, device="cuda")
    C = torch.ones(M, N, dtype=torch.float32, device="cuda")
    dg.sgemm_f32(A, B, C)
    assert bool((C == float(1 + K)).all())


@pytest.mark.parametrize("shape", [(2088, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 512)])
def test_large_sampled(oracle, shape):
    """Large shapes: sampled entries recomputed one by one by the oracle, plus a Freivalds-style
    whole-matrix property in binary64."""
    M, N, K = shape
    rng = _rng(5)
    A, B, C = _draw(rng, (M, K), False), _draw(rng, (K, N), False), _draw(rng, (M, N), False)
    dA, dB, dC = (torch.from_numpy(x).cuda() for x in (A, B, C))
    for rep in range(2):  # the second run adds A B again
        dg.sgemm_f32(dA, dB, dC)
    assert dg.sgemm_last_device_status() == dg.DGEMM_OK
    got = dC.cpu().numpy()
    ii, jj = rng.integers(0, M, 512), rng.integers(0, N, 512)
    once = oracle.sgemm_oracle_entries(A, B, C, ii, jj)
    Cmid = C.copy()
    Cmid[ii, jj] = once
    want = oracle.sgemm_oracle_entries(A, B, Cmid, ii, jj)
    scale = np.abs(C[ii, jj]).astype(np.float64) + 2.0 * np.einsum("sk,ks->s", np.abs(A[ii, :]).astype(np.float64),
                                                                    np.abs(B[:, jj]).astype(np.float64))
    assert (np.abs(got[ii, jj].astype(np.float64) - want.astype(np.float64)) <= 2.0 * (2 * K) * U32 * scale).all()
    x = rng.integers(-1, 2, size=(N, 2)).astype(np.float64)
    lhs = got.astype(np.float64) @ x
    rhs = C.astype(np.float64) @ x + 2.0 * (A.astype(np.float64) @ (B.astype(np.float64) @ x))
    s2 = np.abs(C).astype(np.float64) @ np.abs(x) + 2.0 * (np.abs(A).astype(np.float64) @ (np.abs(B).astype(np.float64) @ np.abs(x)))
    assert (np.abs(lhs - rhs) <= 4.0 * K * U32 * s2).all()


def test_repeated_runs_bit_identical():
    M, N, K = 1536, 1280, 1024
    g = torch.Generator(device="cuda").manual_seed(3)
    A = torch.randint(-4, 5, (M, K), device="cuda", generator=g).float()
    B = torch.randint(-4, 5, (K, N), device="cuda", generator=g).float()
    C0 = torch.randint(-4, 5, (M, N), device="cuda", generator=g).float()
    want = C0.double() + A.double() @ B.double()  # exact in binary64, representable in binary32
    for rep in range(5):
        C = C0.clone()
        dg.sgemm_f32(A, B, C)
        assert torch.equal(C.double(), want), f"run {rep}"
