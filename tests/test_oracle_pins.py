"""Pins for the CPU oracle: each test anchors it to something other than itself.

A plausible mistake anywhere in the oracle (dropped term, wrong sign, transposed operand,
wrong leading dimension, off-by-one loop bound, C ignored or overwritten, reordered sum) fails
at least one of these. CPU only.
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    vals = {}
    with open(os.path.join(HERE, "golden", "paper_worked_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                vals[k] = float(v)
    return vals


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _ints(rng, shape, lo=-4, hi=4):
    return rng.integers(lo, hi + 1, size=shape).astype(np.float64)


def _padded(x, ld, fill=np.nan):
    buf = np.full((x.shape[0], ld), fill)
    buf[:, : x.shape[1]] = x
    return buf, buf[:, : x.shape[1]]


# P1 -- the paper's own driver input: A = B = C = 1 => every entry becomes 1 + K ------------

def test_all_ones_paper_driver(oracle):
    g = _golden()
    K = int(g["all_ones_K"])
    # the paper's operands are 2048 x 2048; rows are independent, so a slab of rows suffices
    M, N = 8, K
    A, B, C = np.ones((M, K)), np.ones((K, N)), np.ones((M, N))
    oracle.dgemm_oracle(A, B, C)
    assert (C == g["all_ones_result"]).all()
    C2 = np.ones((3, 5))
    oracle.dgemm_oracle_ijk(np.ones((3, K)), np.ones((K, 5)), C2)
    assert (C2 == 1.0 + K).all()


# P2 / P3 -- identity and permutation operands: bit-exact for any finite real data -----------

@pytest.mark.parametrize("fn", ["ijk", "ikj"])
def test_identity_and_permutation(oracle, fn):
    run = oracle.dgemm_oracle_ijk if fn == "ijk" else oracle.dgemm_oracle
    rng = _rng(1)
    n, m = 37, 23
    X = rng.uniform(-1, 1, (n, m))
    C0 = rng.uniform(-1, 1, (n, m))
    # A = I  =>  C + B
    C = C0.copy()
    run(np.eye(n), X, C)
    assert np.array_equal(C, C0 + X)
    # B = I  =>  C + A
    Y = rng.uniform(-1, 1, (m, n))
    D0 = rng.uniform(-1, 1, (m, n))
    D = D0.copy()
    run(Y, np.eye(n), D)
    assert np.array_equal(D, D0 + Y)
    # A = row permutation P (P[i, p[i]] = 1)  =>  C[i] + B[p[i]]
    p = rng.permutation(n)
    P = np.zeros((n, n))
    P[np.arange(n), p] = 1.0
    C = C0.copy()
    run(P, X, C)
    assert np.array_equal(C, C0 + X[p])
    # B = P  =>  column j of the product is column q of A where P[q, j] = 1
    D = D0.copy()
    run(Y, P, D)
    inv = np.empty(n, dtype=int)
    inv[p] = np.arange(n)
    assert np.array_equal(D, D0 + Y[:, inv])
    # a non-symmetric permutation distinguishes A@B from B@A, A.T@B and (A@B).T
    assert not np.array_equal(X[p], X[inv])


# P4 -- rank-1 ---------------------------------------------------------------------------------

def test_rank1(oracle):
    rng = _rng(2)
    u, v = rng.uniform(-1, 1, (19, 1)), rng.uniform(-1, 1, (1, 13))
    C = np.zeros((19, 13))
    oracle.dgemm_oracle(u, v, C)
    assert np.array_equal(C, u * v)  # one rounding per entry, fused or not
    # K > 1, constant along k, small integers: C_ij = K * u_i * v_j exactly
    K = 29
    ui, vi = _ints(rng, (19, 1)), _ints(rng, (1, 13))
    C = np.zeros((19, 13))
    oracle.dgemm_oracle_ijk(np.repeat(ui, K, axis=1), np.repeat(vi, K, axis=0), C)
    assert np.array_equal(C, K * ui * vi)


# P5 -- brute force on tiny shapes against an independent int64 accumulation -----------------

def _brute_int(A, B, C):
    M, K = A.shape
    N = B.shape[1]
    out = [[int(C[i][j]) for j in range(N)] for i in range(M)]
    for i in range(M):
        for j in range(N):
            s = 0
            for k in range(K):
                s += int(A[i][k]) * int(B[k][j])
            out[i][j] += s
    return np.array(out, dtype=np.float64).reshape(M, N)


def test_brute_force_tiny_all_shapes(oracle):
    rng = _rng(3)
    dims = [0, 1, 2, 3, 4, 5]
    for M, N, K in itertools.product(dims, dims, dims):
        A, B, C0 = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (M, N), -9, 9)
        want = _brute_int(A, B, C0)
        for run in (oracle.dgemm_oracle_ijk, oracle.dgemm_oracle):
            C = C0.copy()
            run(A, B, C)
            assert np.array_equal(C, want), (M, N, K)


@pytest.mark.parametrize("shape", [(7, 11, 13), (17, 9, 16), (16, 17, 1), (1, 1, 17), (13, 1, 8)])
def test_brute_force_padded_leading_dimensions(oracle, shape):
    M, N, K = shape
    rng = _rng(4)
    A, B, C0 = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (M, N), -9, 9)
    want = _brute_int(A, B, C0)
    Abuf, Av = _padded(A, K + 3)
    Bbuf, Bv = _padded(B, N + 5)
    for run in (oracle.dgemm_oracle_ijk, oracle.dgemm_oracle):
        Cbuf, Cv = _padded(C0, N + 7, fill=-12345.0)
        run(Av, Bv, Cv)
        assert np.array_equal(Cv, want)            # NaN padding of A/B never reaches C
        assert (Cbuf[:, N:] == -12345.0).all()     # P10: padding of C untouched


# P6 -- exact rational arithmetic: the oracle is within the textbook bound of the true value --

def test_exact_rational_within_bound(oracle):
    rng = _rng(5)
    M, N, K = 6, 5, 777
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C = C0.copy()
    oracle.dgemm_oracle(A, B, C)
    u = Fraction(1, 2 ** 53)
    worst = 0.0
    for i in range(M):
        for j in range(N):
            exact = Fraction(C0[i, j])
            scale = abs(Fraction(C0[i, j]))
            for k in range(K):
                exact += Fraction(A[i, k]) * Fraction(B[k, j])
                scale += abs(Fraction(A[i, k]) * Fraction(B[k, j]))
            err = abs(Fraction(C[i, j]) - exact)
            bound = (K + 1) * u * scale  # gamma_{K+1} to first order
            assert err <= bound
            worst = max(worst, float(err / bound))
    assert worst > 0.0  # real data does round; a zero error would mean the test is vacuous


def test_blas_cross_check(oracle):
    """Special case that reduces to a library routine: numpy's BLAS product, within the
    two-sided bound 2*K*u*(|A||B|) (+ the rounding of adding C)."""
    rng = _rng(6)
    M, N, K = 65, 70, 300
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C = C0.copy()
    oracle.dgemm_oracle(A, B, C)
    ref = C0 + A @ B
    scale = np.abs(C0) + np.abs(A) @ np.abs(B)
    assert (np.abs(C - ref) <= 2 * (K + 1) * oracle.U * scale).all()
    # and a transposed or sign-flipped product is far outside it
    assert not (np.abs(C - (C0 + (B.T @ A.T)[:M, :N] if M == N else C0 - A @ B))
                <= 2 * (K + 1) * oracle.U * scale).all()


# P7 -- loop-order identity ----------------------------------------------------------------------

@pytest.mark.parametrize("threads", [1, 3, 0])
def test_ikj_equals_ijk_bitwise(oracle, threads):
    rng = _rng(7)
    M, N, K = 33, 41, 129
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C1, C2 = C0.copy(), C0.copy()
    oracle.dgemm_oracle_ijk(A, B, C1)
    oracle.dgemm_oracle(A, B, C2, threads=threads)
    assert C1.tobytes() == C2.tobytes()


def test_unfused_multiply_add(oracle):
    """The definition rounds the product and the sum separately. Inputs chosen so that a fused
    multiply-add gives a different answer: a*b = 1 - 2^-54 exactly, which rounds to 1.0."""
    a = 1.0 + 2.0 ** -27
    b = 1.0 - 2.0 ** -27
    A, B = np.array([[a]]), np.array([[b]])
    for run in (oracle.dgemm_oracle_ijk, oracle.dgemm_oracle):
        C = np.array([[-1.0]])
        run(A, B, C)
        assert C[0, 0] == 0.0  # fl(a*b) = 1.0 (ties-to-even), then -1 + 1 = 0; fma would give -2^-54
    out = oracle.dgemm_oracle_entries(A, B, np.array([[-1.0]]), [0], [0])
    assert out[0] == 0.0


# P8 -- K-split invariance: bit-exact for the oracle (same operation sequence) -----------------

def test_k_split_invariance(oracle):
    rng = _rng(8)
    M, N, K, K1 = 21, 18, 100, 37
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C1 = C0.copy()
    oracle.dgemm_oracle(A, B, C1)
    C2 = C0.copy()
    oracle.dgemm_oracle(A[:, :K1], B[:K1, :], C2)   # strided views: lda = K
    oracle.dgemm_oracle(A[:, K1:], B[K1:, :], C2)
    assert C1.tobytes() == C2.tobytes()


# P9 -- transpose symmetry and linearity on integer-valued data (exact) ------------------------

def test_transpose_and_linearity(oracle):
    rng = _rng(9)
    M, N, K = 14, 27, 33
    A, B1, B2 = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (K, N))
    C = np.zeros((M, N))
    oracle.dgemm_oracle(A, B1, C)
    Ct = np.zeros((N, M))
    oracle.dgemm_oracle(np.ascontiguousarray(B1.T), np.ascontiguousarray(A.T), Ct)
    assert np.array_equal(C.T, Ct)
    S = np.zeros((M, N))
    oracle.dgemm_oracle(A, B1, S)
    oracle.dgemm_oracle(A, B2, S)            # accumulates: C += uses the incoming C
    L = np.zeros((M, N))
    oracle.dgemm_oracle(A, B1 + B2, L)
    assert np.array_equal(S, L)


# degenerate shapes -------------------------------------------------------------------------------

def test_degenerate_shapes(oracle):
    C0 = np.array([[-0.0, np.nan], [3.5, -1.0]])
    C = C0.copy()
    oracle.dgemm_oracle(np.zeros((2, 0)), np.zeros((0, 2)), C)   # K = 0: C untouched bit for bit
    assert C.tobytes() == C0.tobytes()
    oracle.dgemm_oracle(np.zeros((0, 3)), np.zeros((3, 2)), np.zeros((0, 2)))
    oracle.dgemm_oracle(np.zeros((2, 3)), np.zeros((3, 0)), np.zeros((2, 0)))
    with pytest.raises(ValueError):
        oracle.dgemm_oracle(np.zeros((2, 3)), np.zeros((4, 2)), np.zeros((2, 2)))
    X = np.zeros((4, 4))
    with pytest.raises(ValueError):
        oracle.dgemm_oracle(X, np.zeros((4, 4)), X)              # C aliases A


def test_nan_propagation_row_only(oracle):
    A = np.ones((4, 6))
    A[2, 3] = np.nan
    C = np.zeros((4, 5))
    oracle.dgemm_oracle(A, np.ones((6, 5)), C)
    assert np.isnan(C[2]).all() and np.isfinite(np.delete(C, 2, axis=0)).all()


# sampled entries agree with the full oracle, and the bound scale is |C|+|A||B| ---------------

def test_entries_match_full_and_scale(oracle):
    rng = _rng(10)
    M, N, K = 40, 50, 60
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    Abuf, Av = _padded(A, K + 3)
    Bbuf, Bv = _padded(B, N + 5)
    C = C0.copy()
    oracle.dgemm_oracle(Av, Bv, C)
    ii = rng.integers(0, M, 200)
    jj = rng.integers(0, N, 200)
    got = oracle.dgemm_oracle_entries(Av, Bv, C0, ii, jj)
    assert got.tobytes() == C[ii, jj].tobytes()
    sc = oracle.dgemm_oracle_entries(Av, Bv, C0, ii, jj, absolute=True)
    ref = (np.abs(C0) + np.abs(A) @ np.abs(B))[ii, jj]
    assert np.allclose(sc, ref, rtol=1e-13, atol=0)
    dense = oracle.abs_product(A, B, C0)
    assert dense[ii, jj].tobytes() == sc.tobytes()
    with pytest.raises(IndexError):
        oracle.dgemm_oracle_entries(A, B, None, [M], [0])


# P11 -- Freivalds' check: accepts the oracle's result, rejects a single corrupted entry --------

def test_freivalds_accepts_and_rejects(oracle):
    rng = _rng(11)
    M, N, K = 96, 80, 64
    A, B, C0 = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (M, N))
    C = C0.copy()
    oracle.dgemm_oracle(A, B, C)
    X = oracle.freivalds_vectors(N, 20, seed=5)
    assert set(np.unique(X)) == {-1.0, 1.0}
    resid, _ = oracle.freivalds_residual(A, B, C0, C, X)
    assert (resid == 0).all()                     # integer data: exact
    bad = C.copy()
    bad[17, 3] += 1.0
    resid, _ = oracle.freivalds_residual(A, B, C0, bad, X)
    assert (resid[17] != 0).all() and (np.delete(resid, 17, axis=0) == 0).all()
    # real data: within the rounding tolerance, and a visible perturbation is caught
    A, B, C0 = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C = C0.copy()
    oracle.dgemm_oracle(A, B, C)
    resid, tol = oracle.freivalds_residual(A, B, C0, C, X)
    assert (resid <= tol).all()
    bad = C.copy()
    bad[5, 7] += 1e-9
    resid, tol = oracle.freivalds_residual(A, B, C0, bad, X)
    assert (resid[5] > tol[5]).all()


# the GFLOPS accounting used by the benchmark is the paper's -------------------------------------

def test_gflops_formula_matches_paper():
    g = _golden()
    gf = 2.0 * g["gflops_M"] * g["gflops_N"] * g["gflops_K"] / g["gflops_seconds"] / 1e9
    assert abs(gf - g["gflops_value"]) < 0.005
    assert abs(2 * 4 * 2 * 4.7 - g["peak_gflops"]) < 1e-9


# ---- general form: C = alpha * op(A) op(B) + beta * C (Section 2.15, the options the paper sets aside) ----

def _stored(x, trans):
    """The array as the caller stores it: the transpose (made contiguous) when `trans`."""
    return np.ascontiguousarray(x.T) if trans else x.copy()


@pytest.mark.parametrize("transa,transb", list(itertools.product([False, True], repeat=2)))
def test_general_integer_brute_force(oracle, transa, transb):
    """Python int arithmetic, indices written out from the definition, all four operand forms,
    non-square shapes so that a wrong transpose or leading dimension cannot go unnoticed."""
    rng = _rng(100 + 2 * transa + transb)
    M, N, K = 5, 7, 6
    A, B, C = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (M, N))
    alpha, beta = 3.0, -2.0
    As, Bs = _stored(A, transa), _stored(B, transb)
    bufA, vA = _padded(As, As.shape[1] + 3)
    bufB, vB = _padded(Bs, Bs.shape[1] + 2)
    bufC, vC = _padded(C, N + 5)
    oracle.dgemm_oracle_general(transa, transb, alpha, vA, vB, beta, vC)
    for i in range(M):
        for j in range(N):
            s = 0
            for k in range(K):
                a = int(As[k, i]) if transa else int(As[i, k])
                b = int(Bs[j, k]) if transb else int(Bs[k, j])
                s += a * b
            assert vC[i, j] == 3 * s - 2 * int(C[i, j]), (i, j)
    assert np.isnan(bufC[:, N:]).all() and np.isnan(bufA[:, As.shape[1]:]).all()


def test_general_reduces_to_plain_definition(oracle):
    """alpha = beta = 1, no transposition: bit-identical to the paper's nest started from C
    only when the sum is exact; on real data it differs by the order 'sum then add C', so the
    check is within the bound, and exact on integers."""
    rng = _rng(7)
    M, N, K = 9, 11, 13
    A, B, C = _ints(rng, (M, K)), _ints(rng, (K, N)), _ints(rng, (M, N))
    C1, C2 = C.copy(), C.copy()
    oracle.dgemm_oracle_ijk(A, B, C1)
    oracle.dgemm_oracle_general(False, False, 1.0, A, B, 1.0, C2)
    assert np.array_equal(C1, C2)
    A, B, C = rng.uniform(-1, 1, (M, K)), rng.uniform(-1, 1, (K, N)), rng.uniform(-1, 1, (M, N))
    C1, C2 = C.copy(), C.copy()
    oracle.dgemm_oracle_ijk(A, B, C1)
    oracle.dgemm_oracle_general(False, False, 1.0, A, B, 1.0, C2)
    bound = oracle.entry_bound(K, np.abs(C) + np.abs(A) @ np.abs(B))
    assert (np.abs(C1 - C2) <= bound).all()


def test_general_exact_rationals_within_bound(oracle):
    """Against exact rational arithmetic: |fl - exact| <= (K+2) u (|alpha| |A||B| + |beta||C|)."""
    rng = _rng(11)
    M, N, K = 4, 5, 17
    alpha, beta = 0.3, -1.7
    A, B, C = rng.uniform(-1, 1, (K, M)), rng.uniform(-1, 1, (N, K)), rng.uniform(-1, 1, (M, N))
    out = C.copy()
    oracle.dgemm_oracle_general(True, True, alpha, A, B, beta, out)
    u = Fraction(1, 2 ** 53)
    for i in range(M):
        for j in range(N):
            s = sum(Fraction(A[k, i]) * Fraction(B[j, k]) for k in range(K))
            exact = Fraction(alpha) * s + Fraction(beta) * Fraction(C[i, j])
            scale = abs(Fraction(alpha)) * sum(abs(Fraction(A[k, i]) * Fraction(B[j, k])) for k in range(K)) \
                + abs(Fraction(beta) * Fraction(C[i, j]))
            assert abs(Fraction(out[i, j]) - exact) <= (K + 2) * u * scale * Fraction(101, 100)


def test_general_zero_scalars_do_not_read(oracle):
    """beta == 0: C is output only (NaN in, finite out). alpha == 0: A and B are not read
    (NaN operands leave C = beta*C). K == 0 behaves like alpha == 0."""
    rng = _rng(5)
    M, N, K = 6, 4, 3
    A, B = _ints(rng, (M, K)), _ints(rng, (K, N))
    C = np.full((M, N), np.nan)
    oracle.dgemm_oracle_general(False, False, 2.0, A, B, 0.0, C)
    assert np.array_equal(C, 2.0 * (A @ B))
    C0 = _ints(rng, (M, N))
    C = C0.copy()
    oracle.dgemm_oracle_general(False, False, 0.0, np.full((M, K), np.nan), np.full((K, N), np.nan), 3.0, C)
    assert np.array_equal(C, 3.0 * C0)
    C = C0.copy()
    oracle.dgemm_oracle_general(False, False, 5.0, np.zeros((M, 0)), np.zeros((0, N)), -1.0, C)
    assert np.array_equal(C, -C0)
    C = np.full((M, N), np.nan)
    oracle.dgemm_oracle_general(False, False, 0.0, A, B, 0.0, C)
    assert np.array_equal(C, np.zeros((M, N)))


def test_general_transpose_identity(oracle):
    """(op(A) op(B))^T = op(B)^T op(A)^T: computing C^T with swapped, re-flagged operands gives
    the transposed result exactly on integer data; checked for every operand form."""
    rng = _rng(23)
    M, N, K = 6, 9, 4
    A, B = _ints(rng, (M, K)), _ints(rng, (K, N))
    want = A @ B
    for ta, tb in itertools.product([False, True], repeat=2):
        C = np.zeros((M, N))
        oracle.dgemm_oracle_general(ta, tb, 1.0, _stored(A, ta), _stored(B, tb), 0.0, C)
        assert np.array_equal(C, want), (ta, tb)
        Ct = np.zeros((N, M))  # C^T = B^T A^T: operand "A" is B^T stored as (N x K) or its transpose
        oracle.dgemm_oracle_general(not tb, not ta, 1.0, _stored(B, tb), _stored(A, ta), 0.0, Ct)
        assert np.array_equal(Ct, want.T), (ta, tb)


# ---- binary32 oracle (Section 2.13: the same nest on f32) ------------------------------------------

def _f32(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def test_sgemm_all_ones_driver(oracle):
    """The paper's driver initialises every matrix to one: each entry becomes 1 + K, exact in
    binary32 for K < 2^24."""
    M, N, K = 33, 40, 2048
    A, B, C = np.ones((M, K), np.float32), np.ones((K, N), np.float32), np.ones((M, N), np.float32)
    oracle.sgemm_oracle_ijk(A, B, C)
    assert (C == np.float32(1 + K)).all()
    C2 = np.ones((M, N), np.float32)
    oracle.sgemm_oracle(A, B, C2)
    assert np.array_equal(C, C2)


def test_sgemm_integer_brute_force_and_padding(oracle):
    rng = _rng(41)
    M, N, K = 5, 7, 6
    A, B, C = _f32(_ints(rng, (M, K))), _f32(_ints(rng, (K, N))), _f32(_ints(rng, (M, N)))
    bufA = np.full((M, K + 3), np.nan, np.float32); bufA[:, :K] = A
    bufB = np.full((K, N + 2), np.nan, np.float32); bufB[:, :N] = B
    bufC = np.full((M, N + 5), np.nan, np.float32); bufC[:, :N] = C
    oracle.sgemm_oracle_ijk(bufA[:, :K], bufB[:, :N], bufC[:, :N])
    for i in range(M):
        for j in range(N):
            assert bufC[i, j] == int(C[i, j]) + sum(int(A[i, k]) * int(B[k, j]) for k in range(K))
    assert np.isnan(bufC[:, N:]).all()


def test_sgemm_arithmetic_is_binary32(oracle):
    """2^24 + 1 is not a binary32 number: adding K ones to 2^24 one at a time stays at 2^24 in
    binary32, while any wider accumulator would give 2^24 + K. A product that needs rounding
    pins the multiply as well: (1 + 2^-12)^2 rounds to 1 + 2^-11 in binary32."""
    K = 8
    A, B = np.ones((1, K), np.float32), np.ones((K, 1), np.float32)
    C = np.full((1, 1), 2.0 ** 24, np.float32)
    oracle.sgemm_oracle_ijk(A, B, C)
    assert C[0, 0] == np.float32(2.0 ** 24)
    x = np.float32(1 + 2.0 ** -12)
    C = np.zeros((1, 1), np.float32)
    oracle.sgemm_oracle_ijk(np.array([[x]], np.float32), np.array([[x]], np.float32), C)
    assert C[0, 0] == np.float32(1 + 2.0 ** -11)
    out = oracle.sgemm_oracle_entries(np.array([[x]], np.float32), np.array([[x]], np.float32), None, [0], [0])
    assert out[0] == np.float32(1 + 2.0 ** -11)


def test_sgemm_exact_rationals_within_bound(oracle):
    """|fl32 - exact| <= K u32 (|C| + |A||B|) (1 + small), u32 = 2^-24, against exact rationals."""
    rng = _rng(43)
    M, N, K = 4, 5, 33
    A, B, C = _f32(rng.uniform(-1, 1, (M, K))), _f32(rng.uniform(-1, 1, (K, N))), _f32(rng.uniform(-1, 1, (M, N)))
    out = C.copy()
    oracle.sgemm_oracle(A, B, out)
    u = Fraction(1, 2 ** 24)
    worst = Fraction(0)
    for i in range(M):
        for j in range(N):
            exact = Fraction(float(C[i, j])) + sum(Fraction(float(A[i, k])) * Fraction(float(B[k, j])) for k in range(K))
            scale = abs(Fraction(float(C[i, j]))) + sum(abs(Fraction(float(A[i, k])) * Fraction(float(B[k, j]))) for k in range(K))
            err = abs(Fraction(float(out[i, j])) - exact)
            assert err <= (K + 1) * u * scale * Fraction(101, 100)
            worst = max(worst, err / (u * scale))
    assert worst > Fraction(1, 100)  # binary32 rounding really happened (a binary64 result would be ~1e-9 here)


def test_sgemm_loop_orders_and_entries_agree(oracle):
    rng = _rng(47)
    M, N, K = 37, 29, 101
    A, B, C = _f32(rng.uniform(-1, 1, (M, K))), _f32(rng.uniform(-1, 1, (K, N))), _f32(rng.uniform(-1, 1, (M, N)))
    C1, C2 = C.copy(), C.copy()
    oracle.sgemm_oracle_ijk(A, B, C1)
    oracle.sgemm_oracle(A, B, C2, threads=3)
    assert C1.tobytes() == C2.tobytes()
    ii, jj = rng.integers(0, M, 50), rng.integers(0, N, 50)
    got = oracle.sgemm_oracle_entries(A, B, C, ii, jj)
    assert np.array_equal(got, C1[ii, jj])
    # cross-check with a library routine in higher precision, within the binary32 bound
    ref = C.astype(np.float64) + A.astype(np.float64) @ B.astype(np.float64)
    scale = np.abs(C).astype(np.float64) + np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64)
    assert (np.abs(C1 - ref) <= (K + 1) * oracle.U32 * scale * 1.01).all()
