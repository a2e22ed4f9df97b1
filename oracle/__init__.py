"""CPU oracle for ``C += A @ B`` in IEEE binary64 -- TEST INFRASTRUCTURE ONLY.

This package wraps the plain C triple loop in ``dgemm_oracle.c`` (the paper's naive
three-deep nest, Section 2.1 "Affine Ops"; row-major identity layout, Section 2.2 "MemRefs")
and adds the two verification procedures built on top of it: the per-entry error-bound scale
``(|C|+|A||B|)_ij`` and Freivalds' randomized product check. It is imported only by the
test-suite, by the smoke check and by the benchmark's CPU-baseline leg. It shares no code with
the CUDA library and must never be reachable from the product path.

All pins that anchor it to something other than itself live in ``tests/test_oracle_pins.py``
(closed forms, int64 brute force, exact rational arithmetic, BLAS cross-check, invariants);
nothing here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dgemm_oracle.c")
_HDR = os.path.join(_HERE, "dgemm_oracle.h")
_LIB = os.path.join(_HERE, "libdgemm_oracle.so")
_lock = threading.Lock()
_lib = None

# No reassociation, no fma contraction: the per-element operation sequence is the definition's.
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-std=c99"]


def build(force: bool = False) -> str:
    """Compile the C oracle into ``libdgemm_oracle.so`` next to its source (gcc only)."""
    with _lock:
        stale = (not os.path.exists(_LIB)
                 or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR)))
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.run(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"], check=True, cwd=_HERE)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, dp, ip = ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p
        lib.dgemm_oracle_ijk.argtypes = [i64, i64, i64, dp, i64, dp, i64, dp, i64]
        lib.dgemm_oracle_ijk.restype = None
        lib.dgemm_oracle_ikj.argtypes = [i64, i64, i64, dp, i64, dp, i64, dp, i64, ctypes.c_int]
        lib.dgemm_oracle_ikj.restype = None
        lib.dgemm_oracle_entries.argtypes = [i64, dp, i64, dp, i64, dp, i64, i64, ip, ip,
                                             ctypes.c_int, dp, ctypes.c_int]
        lib.dgemm_oracle_entries.restype = None
        lib.dgemm_oracle_general.argtypes = [ctypes.c_int, ctypes.c_int, i64, i64, i64, ctypes.c_double, dp, i64,
                                             dp, i64, ctypes.c_double, dp, i64, ctypes.c_int]
        lib.dgemm_oracle_general.restype = None
        lib.sgemm_oracle_ijk.argtypes = [i64, i64, i64, dp, i64, dp, i64, dp, i64]
        lib.sgemm_oracle_ijk.restype = None
        lib.sgemm_oracle_ikj.argtypes = [i64, i64, i64, dp, i64, dp, i64, dp, i64, ctypes.c_int]
        lib.sgemm_oracle_ikj.restype = None
        lib.sgemm_oracle_entries.argtypes = [i64, dp, i64, dp, i64, dp, i64, i64, ip, ip, dp, ctypes.c_int]
        lib.sgemm_oracle_entries.restype = None
        lib.dgemm_oracle_max_threads.argtypes = []
        lib.dgemm_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().dgemm_oracle_max_threads())


def _as_np(x) -> np.ndarray:
    """Accept a numpy array or a CPU torch tensor (shared memory, no copy)."""
    if isinstance(x, np.ndarray):
        return x
    if hasattr(x, "detach") and hasattr(x, "numpy"):
        return x.detach().numpy()
    return np.asarray(x)


def _mat(x, name: str, writable: bool = False, dtype=np.float64):
    """Return (array, pointer, rows, cols, ld) for a 2-D float64 matrix with unit column stride.

    A row stride larger than the column count expresses a padded leading dimension (a view
    ``buf[:, :cols]`` of a wider buffer); the padding is never touched.
    """
    a = _as_np(x)
    esz = np.dtype(dtype).itemsize  # float32 matrices for the sgemm functions
    if a.dtype != dtype or a.ndim != 2:
        raise TypeError(f"{name}: need a 2-D {np.dtype(dtype).name} array, got {a.dtype} ndim={a.ndim}")
    rows, cols = a.shape
    if cols > 0 and rows > 0:
        if a.strides[1] != esz:
            raise ValueError(f"{name}: columns must be contiguous (row-major)")
        if rows > 1 and (a.strides[0] % esz != 0 or a.strides[0] < esz * cols):
            raise ValueError(f"{name}: bad row stride {a.strides[0]}")
    if writable and not a.flags.writeable:
        raise ValueError(f"{name}: must be writable")
    ld = a.strides[0] // esz if rows > 1 and cols > 0 else max(cols, 1)
    return a, a.ctypes.data, rows, cols, max(ld, 1)


def _check_shapes(A, B, C):
    a, pa, M, K, lda = _mat(A, "A")
    b, pb, K2, N, ldb = _mat(B, "B")
    c, pc, M2, N2, ldc = _mat(C, "C", writable=True)
    if K != K2 or M != M2 or N != N2:
        raise ValueError(f"shape mismatch: A {a.shape}, B {b.shape}, C {c.shape}")
    if np.shares_memory(c, a) or np.shares_memory(c, b):
        raise ValueError("C must not overlap A or B")
    return (a, b, c), (M, N, K, pa, lda, pb, ldb, pc, ldc)


def dgemm_oracle_ijk(A, B, C) -> None:
    """In place ``C += A @ B`` by the definition (loops i, j, k; multiply then add)."""
    keep, args = _check_shapes(A, B, C)
    _load().dgemm_oracle_ijk(*args)
    del keep


def dgemm_oracle(A, B, C, threads: int = 0) -> None:
    """In place ``C += A @ B``, loop order i, k, j over OpenMP rows; bit-identical to the definition."""
    keep, args = _check_shapes(A, B, C)
    _load().dgemm_oracle_ikj(*args, int(threads))
    del keep


def dgemm_oracle_general(transa: bool, transb: bool, alpha: float, A, B, beta: float, C, threads: int = 0) -> None:
    """In place ``C = alpha * op(A) @ op(B) + beta * C`` by the definition. ``A`` is given as stored
    (K x M when ``transa``), likewise ``B`` (N x K when ``transb``)."""
    a, pa, ar, ac, lda = _mat(A, "A")
    b, pb, br, bc, ldb = _mat(B, "B")
    c, pc, M, N, ldc = _mat(C, "C", writable=True)
    Ma, K = (ac, ar) if transa else (ar, ac)
    K2, Nb = (bc, br) if transb else (br, bc)
    if K != K2 or Ma != M or Nb != N:
        raise ValueError(f"shape mismatch: A {a.shape} (transa={transa}), B {b.shape} (transb={transb}), C {c.shape}")
    if np.shares_memory(c, a) or np.shares_memory(c, b):
        raise ValueError("C must not overlap A or B")
    _load().dgemm_oracle_general(int(bool(transa)), int(bool(transb)), M, N, K, float(alpha), pa, lda, pb, ldb,
                                 float(beta), pc, ldc, int(threads))


def dgemm_oracle_entries(A, B, Cin, ii, jj, absolute: bool = False, threads: int = 0) -> np.ndarray:
    """Entries ``(Cin + A @ B)[ii[s], jj[s]]`` recomputed one by one with the definition's k loop.

    ``Cin`` may be ``None`` (zero). With ``absolute=True`` the magnitudes of all operands are
    used, which gives the scale ``(|Cin| + |A||B|)_ij`` of the per-entry error bound.
    """
    a, pa, M, K, lda = _mat(A, "A")
    b, pb, K2, N, ldb = _mat(B, "B")
    if K != K2:
        raise ValueError("shape mismatch")
    pc, ldc, c = None, 1, None
    if Cin is not None:
        c, pc, M2, N2, ldc = _mat(Cin, "Cin")
        if (M2, N2) != (M, N):
            raise ValueError("shape mismatch")
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    if ii.shape != jj.shape or ii.ndim != 1:
        raise ValueError("ii, jj must be 1-D of equal length")
    if ii.size and (ii.min() < 0 or ii.max() >= M or jj.min() < 0 or jj.max() >= N):
        raise IndexError("sample index out of range")
    out = np.empty(ii.size, dtype=np.float64)
    _load().dgemm_oracle_entries(K, pa, lda, pb, ldb, pc, ldc, ii.size, ii.ctypes.data,
                                 jj.ctypes.data, int(bool(absolute)), out.ctypes.data, int(threads))
    del a, b, c
    return out


def _check_shapes_f32(A, B, C):
    a, pa, M, K, lda = _mat(A, "A", dtype=np.float32)
    b, pb, K2, N, ldb = _mat(B, "B", dtype=np.float32)
    c, pc, M2, N2, ldc = _mat(C, "C", writable=True, dtype=np.float32)
    if K != K2 or M != M2 or N != N2:
        raise ValueError(f"shape mismatch: A {a.shape}, B {b.shape}, C {c.shape}")
    if np.shares_memory(c, a) or np.shares_memory(c, b):
        raise ValueError("C must not overlap A or B")
    return (a, b, c), (M, N, K, pa, lda, pb, ldb, pc, ldc)


def sgemm_oracle_ijk(A, B, C) -> None:
    """In place ``C += A @ B`` in binary32 by the definition (loops i, j, k; multiply then add)."""
    keep, args = _check_shapes_f32(A, B, C)
    _load().sgemm_oracle_ijk(*args)
    del keep


def sgemm_oracle(A, B, C, threads: int = 0) -> None:
    """In place binary32 ``C += A @ B``, loops i, k, j over OpenMP rows; bit-identical to the definition."""
    keep, args = _check_shapes_f32(A, B, C)
    _load().sgemm_oracle_ikj(*args, int(threads))
    del keep


def sgemm_oracle_entries(A, B, Cin, ii, jj, threads: int = 0) -> np.ndarray:
    """Binary32 entries ``(Cin + A @ B)[ii[s], jj[s]]`` recomputed one by one (``Cin`` may be None)."""
    a, pa, M, K, lda = _mat(A, "A", dtype=np.float32)
    b, pb, K2, N, ldb = _mat(B, "B", dtype=np.float32)
    if K != K2:
        raise ValueError("shape mismatch")
    pc, ldc, c = None, 1, None
    if Cin is not None:
        c, pc, M2, N2, ldc = _mat(Cin, "Cin", dtype=np.float32)
        if (M2, N2) != (M, N):
            raise ValueError("shape mismatch")
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    if ii.shape != jj.shape or ii.ndim != 1:
        raise ValueError("ii, jj must be 1-D of equal length")
    if ii.size and (ii.min() < 0 or ii.max() >= M or jj.min() < 0 or jj.max() >= N):
        raise IndexError("sample index out of range")
    out = np.empty(ii.size, dtype=np.float32)
    _load().sgemm_oracle_entries(K, pa, lda, pb, ldb, pc, ldc, ii.size, ii.ctypes.data, jj.ctypes.data,
                                 out.ctypes.data, int(threads))
    del a, b, c
    return out


U32 = 2.0 ** -24  # unit roundoff of binary32


def abs_product(A, B, Cin=None, threads: int = 0) -> np.ndarray:
    """Dense ``|Cin| + |A| @ |B|`` (the error-bound scale), computed with the oracle itself."""
    a, b = np.abs(_as_np(A)), np.abs(_as_np(B))
    s = np.zeros((a.shape[0], b.shape[1])) if Cin is None else np.abs(_as_np(Cin)).copy()
    dgemm_oracle(np.ascontiguousarray(a), np.ascontiguousarray(b), s, threads)
    return s


U = 2.0 ** -53  # unit roundoff of binary64


def entry_bound(K: int, scale):
    """Pass criterion for real-valued data: ``|dC_ij| <= 2*K*2^-53 * scale_ij``.

    Both the oracle and any other correct evaluation order (fused or not) err by at most
    gamma_K * (|A||B|)_ij from the exact sum (standard inner-product bound), so two correct
    results differ by at most twice that.
    """
    return 2.0 * K * U * np.asarray(scale)


def freivalds_vectors(N: int, nvec: int, seed: int) -> np.ndarray:
    """``nvec`` random +-1 column vectors of length N as an (N, nvec) float64 array."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, 2, size=(N, nvec)).astype(np.float64) * 2.0 - 1.0


def freivalds_residual(A, B, Cin, Cout, X):
    """Freivalds' check of ``Cout == Cin + A @ B`` against +-1 vectors ``X`` (N x nvec).

    Returns ``(resid, tol)`` of shape (M, nvec): ``resid = |Cout X - (Cin X + A (B X))|`` and a
    rigorous rounding tolerance for real data,
    ``tol_i = (2K + 2N + 4) * 2^-53 * (sum_j |Cin_ij| + sum_j|Cout_ij| + (|A| (|B| 1))_i)``.
    A wrong ``Cout`` escapes one vector with probability <= 1/2, hence <= 2^-nvec overall. On
    integer-valued data with all partial sums below 2^53 the tolerance can be taken as zero.
    The mat-vec products are library primitives (numpy), evaluated in float64.
    """
    a, b, cin, cout = _as_np(A), _as_np(B), _as_np(Cin), _as_np(Cout)
    K, N = b.shape
    bx = b @ X
    lhs = cout @ X
    rhs = cin @ X + a @ bx
    resid = np.abs(lhs - rhs)
    ones = np.ones((N, 1))
    scale = (np.abs(cin) @ ones + np.abs(cout) @ ones + np.abs(a) @ (np.abs(b) @ ones))
    tol = (2 * K + 2 * N + 4) * U * scale
    return resid, np.broadcast_to(tol, resid.shape)
