"""Tile-parameter exploration for ``dgemm_f64``: an analytical time model and an autotuner.

The paper explores its tile parameters (M_C, K_C, M_R, N_R, K_U) by recompiling one variant per
point and reasons about the register budget with a small model (Section 2.10, "Tweaking M_C, K_C,
M_R, N_R to maximize reuse"; Section 2.15 points to analytical modelling for choosing them). Here
the points of the space are kernels that are all compiled into the library (a variant table):

    ws128    warp-specialised, 128 x 128 CTA tile, one CTA per SM, software-pipelined consumers
    ws64     the same kernel with 64 x 128 tiles, two CTAs per SM
    inline64 inline load stream, 64 x 128 tiles, two CTAs per SM
    inline128 inline load stream, 128 x 128 tiles, one CTA per SM
    small_wt 128 x 128 tiles built from 32 x 32 warp tiles (16 warps)
    generic  8-byte asynchronous copies instead of TMA (any alignment)
    cluster  64 x 128 tiles, K cut over the CTAs of a thread-block cluster, partial tiles added
             through distributed shared memory (one launch; what the library uses below one wave)
    bulk     warp-specialised, 128 x 128 tiles, five stages, accumulators leave through a shared-memory
             tile buffer and the copy engine's bulk reduce into C (what the library uses for many
             tiles of few k-blocks)

``model_ms`` predicts the time of each from the shape (waves of tiles, a K split of the last
partial wave, the per-tile C round trip, launch latencies); ``autotune`` measures them through the
C ABI and ranks them. Nothing here is on the product path: the library's own choice
(``DGEMM_VARIANT_AUTO``) is fixed in C; this module is how that choice was explored and how it can
be checked on another shape.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional

SM_COUNT = 148
PEAK_TFLOPS = 148 * 64 * 2 * 1.965e9 / 1e12  # FP64 tensor pipe: 64 FMA/clk/SM
HBM_GBS = 6500.0
LAUNCH_US = 3.0        # launch + first copies in flight, measured on small problems (programmatic dependent launch)
REDUCE_US = 4.0        # second launch and the partial-tile reduction when K is split
BK = 16


@dataclass(frozen=True)
class Config:
    name: str
    variant: int          # DGEMM_VARIANT_*
    flags: int            # dgemm_set_test_flags bits
    bm: int
    bn: int
    ctas_per_sm: int
    mainloop_eff: float   # fraction of the pipe peak the steady-state k loop sustains (measured, long K)
    needs_tma: bool = True
    epilogue_exposed: float = -1.0  # share of a tile's C round trip the arithmetic waits for (-1: by CTAs per SM)


CONFIGS: Dict[str, Config] = {
    # epilogue_exposed from the rank-k K = 64 shape (16384^2 x 64: 1516, 1256 and 1354 us measured)
    "ws128": Config("ws128", 3, 0, 128, 128, 1, 0.975, epilogue_exposed=0.86),
    "ws64": Config("ws64", 3, 32, 64, 128, 2, 0.950, epilogue_exposed=0.85),
    "inline64": Config("inline64", 1, 0, 64, 128, 2, 0.970, epilogue_exposed=1.2),
    "inline128": Config("inline128", 1, 4, 128, 128, 1, 0.960),
    "small_wt": Config("small_wt", 1, 4 | 8, 128, 128, 1, 0.945),
    "generic": Config("generic", 2, 16, 64, 128, 2, 0.880, needs_tma=False),
    "cluster": Config("cluster", 5, 0, 64, 128, 2, 0.775),
    # C never enters the SM; what the arithmetic waits for is its own stores into the tile buffer
    "bulk": Config("bulk", 10, 0, 128, 128, 1, 0.955, epilogue_exposed=0.08),
}

KBLOCK_ALONE_US = 1.35   # one k-block of a 64 x 128 tile on an SM the CTA has to itself (measured, long K)
KBLOCK_SHARED_US = 2.2   # the same with a second CTA on the SM
CLUSTER_FIXED_US = 4.0   # first copies, two cluster barriers, exit (128^3: 8.8 us per call in a stream)
CLUSTER_PASS_US = 0.4    # one pass of the in-cluster reduction (512 element pairs per CTA)


def cluster_size(M: int, N: int, K: int) -> int:
    """Cluster size of the forced cluster variant: the largest of 1, 2, 4, 8 that keeps all CTAs
    resident at once and gives every CTA a k-block."""
    tiles, kb = math.ceil(M / 64) * math.ceil(N / 128), math.ceil(K / BK)
    s = 1
    while s < 8 and 2 * s <= kb and tiles * 2 * s <= 2 * SM_COUNT:
        s *= 2
    return s


def model_cluster_ms(M: int, N: int, K: int) -> float:
    tiles, kb = math.ceil(M / 64) * math.ceil(N / 128), math.ceil(K / BK)
    s = cluster_size(M, N, K)
    ctas = tiles * s
    waves = math.ceil(ctas / (2 * SM_COUNT))
    per_kb = KBLOCK_SHARED_US if ctas > SM_COUNT else KBLOCK_ALONE_US
    t = waves * (math.ceil(kb / s) * per_kb + (8 // s) * CLUSTER_PASS_US) + CLUSTER_FIXED_US + LAUNCH_US
    t_pipe = 2.0 * M * N * K / (PEAK_TFLOPS * 1e12) * 1e6
    t_hbm = 8.0 * (M * K + K * N + 2.0 * M * N) / (HBM_GBS * 1e9) * 1e6
    return max(t, t_pipe, t_hbm) * 1e-3


def register_budget(bm: int, bn: int, warps: int, wt_m: int = 64, wt_n: int = 32) -> dict:
    """The register-file arithmetic behind the tile sizes (the analogue of the paper's count of
    vector registers for its M_R x N_R register tile): accumulators + two half-k-block fragment
    sets per thread against the 255-register limit, and the CTA total against the 64 K registers
    of an SM."""
    acc = wt_m * wt_n * 2 // 32                      # 32-bit registers per thread for the FP64 accumulators
    frag = ((wt_m // 16) * 4 + 8) * 2                # one half k-block: A (lo, hi per 16 rows) + B, as doubles
    per_thread = acc + 2 * frag + 24                 # two fragment sets (software pipeline) + addressing
    assert (bm // wt_m) * (bn // wt_n) == warps
    return {"accumulators": acc, "fragments_per_half_kblock": frag, "per_thread": per_thread,
            "fits_255": per_thread <= 255, "cta_registers": per_thread * warps * 32}


def model_ms(M: int, N: int, K: int, cfg: Config, ldc_aligned: bool = True) -> float:
    """Predicted duration of one dgemm_f64 call in milliseconds.

    Time = launch + (k-block iterations per CTA slot) x (time of one k-block at the config's
    steady-state efficiency) + exposed C round trips + the reduction pass when tiles are split.
    Whole waves run data-parallel; the last partial wave is spread evenly (stream-K), as the
    library does."""
    if cfg.name == "cluster":
        return model_cluster_ms(M, N, K)
    tiles_m, tiles_n = math.ceil(M / cfg.bm), math.ceil(N / cfg.bn)
    tiles = tiles_m * tiles_n
    kblocks = math.ceil(K / BK)
    slots = SM_COUNT * cfg.ctas_per_sm
    full_waves = tiles // slots
    tail_tiles = tiles - full_waves * slots
    iters = full_waves * kblocks                       # k-block iterations on the critical CTA
    split = False
    if tail_tiles:
        per_cta = math.ceil(tail_tiles * kblocks / slots)
        if (1.0 - tail_tiles / slots) * kblocks >= 5 and kblocks >= 2:
            iters += per_cta
            split = per_cta < kblocks
        else:
            iters += kblocks
    # one k-block of a bm x bn tile on an SM shared by ctas_per_sm CTAs
    flop_kb = 2.0 * cfg.bm * cfg.bn * BK
    sm_rate = PEAK_TFLOPS * 1e12 / SM_COUNT * cfg.mainloop_eff / cfg.ctas_per_sm
    t_main = iters * flop_kb / sm_rate
    # C round trip per tile: hidden behind the other CTA's arithmetic when two share an SM
    tile_bytes = 2.0 * cfg.bm * cfg.bn * 8
    per_sm_bw = HBM_GBS * 1e9 / SM_COUNT * (1.0 if ldc_aligned else 0.5)
    exposed = cfg.epilogue_exposed if cfg.epilogue_exposed >= 0 else (1.0 if cfg.ctas_per_sm == 1 else 0.35)
    tiles_per_slot = math.ceil(tiles / slots)
    t_epi = tiles_per_slot * tile_bytes / per_sm_bw * exposed
    # the whole problem cannot beat its compulsory HBM traffic
    t_hbm = 8.0 * (M * K + K * N + 2.0 * M * N) / (HBM_GBS * 1e9)
    t = max(t_main + t_epi, t_hbm) + LAUNCH_US * 1e-6 + (REDUCE_US * 1e-6 if split else 0.0)
    return t * 1e3


def predict(M: int, N: int, K: int, tma_ok: bool = True) -> List[dict]:
    """All configurations ranked by the model."""
    rows = []
    for cfg in CONFIGS.values():
        if cfg.needs_tma and not tma_ok:
            continue
        ms = model_ms(M, N, K, cfg)
        rows.append({"config": cfg.name, "model_ms": ms, "model_tflops": 2.0 * M * N * K / ms / 1e9})
    return sorted(rows, key=lambda r: r["model_ms"])


def _time_call(torch, call, reps_ms: float = 30.0) -> float:
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(2):
        call()
    e0.record()
    call()
    e1.record()
    torch.cuda.synchronize()
    reps = int(max(3, min(200, reps_ms / max(e0.elapsed_time(e1), 1e-3))))
    best = float("inf")
    for _ in range(3):
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / reps)
    return best


def autotune(M: int, N: int, K: int, lda: Optional[int] = None, ldb: Optional[int] = None, ldc: Optional[int] = None,
             seed: int = 0) -> List[dict]:
    """Times every applicable configuration (and the library's own choice) on a synthetic problem
    of this shape on the current CUDA device, through the C ABI. Returns rows sorted by measured
    time, each with the model's prediction beside it. Restores the library's settings."""
    import torch

    from . import binding as b

    lda, ldb, ldc = lda or K, ldb or N, ldc or N
    g = torch.Generator(device="cuda").manual_seed(seed)
    A = torch.rand(M, lda, dtype=torch.float64, device="cuda", generator=g) * 2 - 1
    B = torch.rand(K, ldb, dtype=torch.float64, device="cuda", generator=g) * 2 - 1
    C = torch.zeros(M, ldc, dtype=torch.float64, device="cuda")
    pa, pb, pc = A.data_ptr(), B.data_ptr(), C.data_ptr()
    tma_ok = pa % 16 == 0 and pb % 16 == 0 and lda % 2 == 0 and ldb % 2 == 0
    lib = b.load_library()
    rows = []
    try:
        candidates = [("auto", b.DGEMM_VARIANT_AUTO, 0, None)] + [
            (c.name, c.variant, c.flags, c) for c in CONFIGS.values() if tma_ok or not c.needs_tma]
        for name, variant, flags, cfg in candidates:
            b.dgemm_set_variant(variant)
            b.dgemm_set_test_flags(flags)
            rc = lib.dgemm_f64(M, N, K, pa, lda, pb, ldb, pc, ldc, None)
            if rc != 0:
                continue
            ms = _time_call(torch, lambda: lib.dgemm_f64(M, N, K, pa, lda, pb, ldb, pc, ldc, None))
            row = {"config": name, "ms": ms, "tflops": 2.0 * M * N * K / ms / 1e9}
            if cfg is not None:
                row["model_ms"] = model_ms(M, N, K, cfg, ldc_aligned=(ldc % 4 == 0))
            rows.append(row)
    finally:
        b.dgemm_set_variant(b.DGEMM_VARIANT_AUTO)
        b.dgemm_set_test_flags(0)
    assert b.dgemm_last_device_status() == 0
    return sorted(rows, key=lambda r: r["ms"])


if __name__ == "__main__":
    import json
    import sys

    shape = tuple(int(x) for x in sys.argv[1].split(",")) if len(sys.argv) > 1 else (4096, 4096, 4096)
    print(json.dumps({"shape": shape, "ranking": autotune(*shape), "model": predict(*shape),
                      "register_budget_64x32_warp_tile": register_budget(128, 128, 8)}, indent=1))
