"""Randomised parity: random shapes, paddings, base offsets, entry points (dgemm_f64, dgemm_f64_ex,
sgemm_f32), kernel variants and test flags on integer-valued data, where every evaluation order is
exact: sampled entries against the oracle's definition bit for bit, plus row and column sums over
the whole result. Seeded; needs a B200."""
import random

import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg

pytestmark = pytest.mark.gpu


def _dim(rnd, hi):
    r = rnd.random()
    if r < 0.15:
        return rnd.randint(1, 40)
    if r < 0.5:
        return rnd.randint(1, 300)
    return rnd.randint(1, hi)


def _padded(x, pad, off, ttype):
    rows, cols = x.shape
    whole = torch.full((rows * (cols + pad) + off + 8,), float("nan"), dtype=ttype, device="cuda")
    buf = whole[off:off + rows * (cols + pad)].view(rows, cols + pad)
    buf[:, :cols] = torch.from_numpy(x).cuda()
    return buf, buf[:, :cols]


@pytest.mark.parametrize("seed", range(8))
def test_random_cases(oracle, seed):
    rnd = random.Random(seed)
    rng = np.random.Generator(np.random.PCG64(seed))
    for case in range(40):
        M, N, K = _dim(rnd, 1500), _dim(rnd, 1500), _dim(rnd, 2000)
        kind = rnd.choice(["d", "d", "d", "ex", "s"])
        ntype, ttype = (np.float32, torch.float32) if kind == "s" else (np.float64, torch.float64)
        ta = tb = False
        alpha = beta = 1.0
        if kind == "ex":
            ta, tb = rnd.random() < 0.5, rnd.random() < 0.5
            alpha, beta = rnd.choice([(1.0, 1.0), (2.0, -1.0), (-3.0, 0.0), (1.0, 0.0), (0.0, 2.0)])
        A = rng.integers(-3, 4, (K, M) if ta else (M, K)).astype(ntype)
        B = rng.integers(-3, 4, (N, K) if tb else (K, N)).astype(ntype)
        C = rng.integers(-3, 4, (M, N)).astype(ntype)
        pads = [rnd.choice([0, 0, 1, 2, 3, 5]) for _ in range(3)]
        offs = [rnd.choice([0, 0, 0, 1, 2, 3]) for _ in range(3)]
        (_, dA), (_, dB), (bufC, dC) = (_padded(x, p, o, ttype) for x, p, o in zip((A, B, C), pads, offs))
        variant, flags, split = dg.DGEMM_VARIANT_AUTO, 0, 0
        if kind != "s" and rnd.random() < 0.3:
            variant = rnd.choice([1, 2, 3, 4, 5, 6, 7, 8, 9, 10])  # every pipelined kernel, the ladder rungs, the cluster and bulk-epilogue kernels
            flags = rnd.choice([0, 0, 1, 2, 4, 8, 12, 32, 128])
            if rnd.random() < 0.2:
                split = rnd.choice([2, 3, 5])
        what = f"seed {seed} case {case}: {kind} {(M, N, K)} ta={ta} tb={tb} alpha={alpha} beta={beta} pads={pads} " \
               f"offs={offs} variant={variant} flags={flags} split={split}"
        try:
            if kind == "s":
                dg.sgemm_f32(dA, dB, dC)
                assert dg.sgemm_last_device_status() == dg.DGEMM_OK, what
            else:
                dg.dgemm_set_variant(variant)
                dg.dgemm_set_test_flags(flags)
                dg.dgemm_set_split_k(split)
                if kind == "d":
                    rc = dg.dgemm_f64(dA, dB, dC, check=False)
                else:
                    rc = dg.dgemm_f64_ex(dA, dB, dC, alpha=alpha, beta=beta, transa=ta, transb=tb, check=False)
                if rc == dg.binding.DGEMM_ERR_VARIANT:
                    continue  # a forced TMA variant on operands (or a C, a beta) it cannot take, or scalars on a ladder rung
                assert rc == dg.DGEMM_OK, what
                assert dg.dgemm_last_device_status() == dg.DGEMM_OK, what
        finally:
            dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
            dg.dgemm_set_test_flags(0)
            dg.dgemm_set_split_k(0)
        got = dC.cpu().numpy()
        if pads[2]:
            assert bool(torch.isnan(bufC[:, N:]).all()), what
        # sampled entries by the oracle's definition
        n = min(400, M * N)
        ii, jj = rng.integers(0, M, n), rng.integers(0, N, n)
        if kind == "s":
            want = oracle.sgemm_oracle_entries(A, B, C, ii, jj)
        elif kind == "d":
            want = oracle.dgemm_oracle_entries(A, B, C, ii, jj)
        else:
            opA = np.ascontiguousarray(A.T) if ta else A
            opB = np.ascontiguousarray(B.T) if tb else B
            s = oracle.dgemm_oracle_entries(opA, opB, None, ii, jj) if alpha != 0.0 else np.zeros(n)
            want = alpha * s + (beta * C[ii, jj] if beta != 0.0 else 0.0)  # exact: small integers
        assert np.array_equal(got[ii, jj], want), what
        # whole result: row and column sums (exact on this data)
        a64 = (A.T if ta else A).astype(np.float64)
        b64 = (B.T if tb else B).astype(np.float64)
        c64, g64 = C.astype(np.float64), got.astype(np.float64)
        cpart = beta * c64 if beta != 0.0 else np.zeros_like(c64)
        assert np.array_equal(g64.sum(axis=1), cpart.sum(axis=1) + alpha * (a64 @ b64.sum(axis=1))), what
        assert np.array_equal(g64.sum(axis=0), cpart.sum(axis=0) + alpha * (a64.sum(axis=0) @ b64)), what
