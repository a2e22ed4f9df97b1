"""Seeded synthetic inputs for ``C += A @ B`` (FP64, row-major, padded leading dimensions).

This module only *generates data*: it contains none of the method's arithmetic, so both the
CUDA library's tests/benchmark and the CPU oracle's tests may use it without coupling them.

Recipe (the paper's own workload is synthetic dense f64 matrices, Section 2.1; its size sweep
is square): values uniform in [-1, 1) drawn as ``rand * 2 - 1`` (exact in binary64), or uniform
integers in {-4, ..., 4} for the bit-exact mode; one ``torch.Generator`` per problem seeded
with ``seed``; draw order A, then B, then C, each in logical row-major order. The logical
matrices are then placed into ``rows x ld`` buffers whose padding columns are poisoned: NaN
for A and B (a library that reads padding into the result is caught), a recognisable bit
pattern for C (a library that writes padding is caught).
"""
from __future__ import annotations

import dataclasses
import struct
from typing import Optional

import torch

#: Bit pattern written into the padding columns of C (a quiet NaN with a recognisable payload).
C_CANARY_BITS = 0x7FF8_DEAD_BEEF_CAFE
C_CANARY = struct.unpack("<d", struct.pack("<Q", C_CANARY_BITS))[0]


@dataclasses.dataclass
class Problem:
    """One GEMM problem on the host. ``*_buf`` are the padded ``rows x ld`` buffers; ``A``, ``B``,
    ``C`` are the logical views ``buf[:, :cols]`` (they share storage with the buffers)."""
    M: int
    N: int
    K: int
    lda: int
    ldb: int
    ldc: int
    A_buf: torch.Tensor
    B_buf: torch.Tensor
    C_buf: torch.Tensor
    seed: int
    integer: bool

    @property
    def A(self) -> torch.Tensor:
        return self.A_buf[:, : self.K]

    @property
    def B(self) -> torch.Tensor:
        return self.B_buf[:, : self.N]

    @property
    def C(self) -> torch.Tensor:
        return self.C_buf[:, : self.N]

    @property
    def flop(self) -> float:
        return 2.0 * self.M * self.N * self.K

    @property
    def min_bytes(self) -> float:
        """Compulsory HBM traffic: read A, B and C once, write C once."""
        return 8.0 * (self.M * self.K + self.K * self.N + 2 * self.M * self.N)


def _draw(rows: int, cols: int, g: torch.Generator, integer: bool) -> torch.Tensor:
    if integer:
        return torch.randint(-4, 5, (rows, cols), generator=g, dtype=torch.int64).to(torch.float64)
    return torch.rand((rows, cols), generator=g, dtype=torch.float64).mul_(2.0).sub_(1.0)


def _place(x: torch.Tensor, ld: int, fill: float, pin: bool) -> torch.Tensor:
    rows, cols = x.shape
    if ld == cols:
        buf = x.contiguous()
    else:
        buf = torch.full((rows, ld), fill, dtype=torch.float64)
        buf[:, :cols] = x
    return buf.pin_memory() if pin and torch.cuda.is_available() else buf


def make_problem(M: int, N: int, K: int, seed: int, *, lda: Optional[int] = None,
                 ldb: Optional[int] = None, ldc: Optional[int] = None, integer: bool = False,
                 c_zero: bool = False, pin: bool = False) -> Problem:
    """Generate one problem. ``ld*`` default to the logical column counts (dense)."""
    lda = max(K, 1) if lda is None else lda
    ldb = max(N, 1) if ldb is None else ldb
    ldc = max(N, 1) if ldc is None else ldc
    if lda < max(K, 1) or ldb < max(N, 1) or ldc < max(N, 1):
        raise ValueError("leading dimension smaller than the row length")
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    A = _draw(M, K, g, integer)
    B = _draw(K, N, g, integer)
    C = torch.zeros((M, N), dtype=torch.float64) if c_zero else _draw(M, N, g, integer)
    nan = float("nan")
    return Problem(M, N, K, lda, ldb, ldc,
                   _place(A, lda, nan, pin), _place(B, ldb, nan, pin), _place(C, ldc, C_CANARY, pin),
                   seed, integer)


def c_padding_intact(C_buf: torch.Tensor, N: int) -> bool:
    """True iff every padding column of a C buffer still holds the canary bit pattern."""
    if C_buf.shape[1] == N:
        return True
    pad = C_buf[:, N:].contiguous().view(torch.int64)
    want = C_CANARY_BITS - (1 << 64) if C_CANARY_BITS >= (1 << 63) else C_CANARY_BITS
    return bool((pad == want).all())


# --- The five benchmark/parity configurations ------------------------------------------------

def config1(integer: bool) -> Problem:
    """256^3, seed 0, C = 0; real-valued or integer-valued {-4..4}."""
    return make_problem(256, 256, 256, 0, integer=integer, c_zero=True)


def config2_sizes():
    """Square sweep M=N=K = 128, 256, ..., 4096; seed = size; dense leading dimensions."""
    return list(range(128, 4096 + 1, 128))


def config2(n: int, pin: bool = False) -> Problem:
    return make_problem(n, n, n, n, pin=pin)


def config3(integer: bool = False, pin: bool = False) -> Problem:
    """8192^3, seed 1, C random."""
    return make_problem(8192, 8192, 8192, 1, integer=integer, pin=pin)


CONFIG4_SHAPES = [(1000, 1537, 777), (2088, 2088, 2088), (4097, 31, 4099)]


def config4(idx: int) -> Problem:
    """Ragged shapes with padded leading dimensions lda=K+3, ldb=N+5, ldc=N+7; seed 2."""
    M, N, K = CONFIG4_SHAPES[idx]
    return make_problem(M, N, K, 2, lda=K + 3, ldb=N + 5, ldc=N + 7)


CONFIG5_K = [64, 256]


def config5(K: int, pin: bool = False) -> Problem:
    """Rank-k update, M=N=16384, K in {64, 256}; seed 3."""
    return make_problem(16384, 16384, K, 3, pin=pin)


def sample_indices(M: int, N: int, count: int, seed: int, tile: int = 128):
    """``count`` entry positions: forced corners, both sides of several tile boundaries, and
    seeded uniform positions for the rest. Returns two int64 tensors (rows, cols)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    forced = []
    edge_r = sorted({0, M - 1, *[r for t in (1, 2, M // tile) for r in (t * tile - 1, t * tile) if 0 <= r < M]})
    edge_c = sorted({0, N - 1, *[c for t in (1, 2, N // tile) for c in (t * tile - 1, t * tile) if 0 <= c < N]})
    for r in edge_r:
        for c in edge_c:
            forced.append((r, c))
    forced = forced[:count]
    rest = count - len(forced)
    ii = torch.randint(0, M, (rest,), generator=g, dtype=torch.int64)
    jj = torch.randint(0, N, (rest,), generator=g, dtype=torch.int64)
    if forced:
        fi = torch.tensor([f[0] for f in forced], dtype=torch.int64)
        fj = torch.tensor([f[1] for f in forced], dtype=torch.int64)
        ii, jj = torch.cat([fi, ii]), torch.cat([fj, jj])
    return ii, jj
