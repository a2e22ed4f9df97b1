#!/usr/bin/env python
"""Benchmark of libdgemm's hot path: FP64 ``C += A @ B`` at M=N=K=8192 on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--size n]

One step = one ``dgemm_f64`` call (the whole hot path: dispatch, tile schedule, staging, DMMA
main loop, C += epilogue) on one seeded synthetic problem whose operands are resident in HBM.
The headline workload is the large square case (8192^3, uniform [-1,1), seed 1); 1.6 GB of
operands per step exceed the 126 MB L2, so no explicit L2 flush is needed between steps.
Multi-GPU runs are independent replicas (the path has no exchange step): every rank runs the
same problem on its own GPU, the timed region is bracketed by a barrier and a device
synchronisation on both sides, and the reported time is the maximum over ranks.

Prints one JSON line (rank 0 only). ``--impl reference`` times the CPU oracle instead, on a
bounded row slab of the same workload, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

SM_COUNT_B200 = 148
FMA_PER_CLK_SM = 64  # FP64 DMMA issue rate measured by dgemm_fp64_peak_probe (63.95 on B200)

# DRAM traffic of one 8192^3 launch of the dominant kernel (dram__bytes_read.sum +
# dram__bytes_write.sum of one ncu capture, see profiles/); None until a capture exists for a size.
NCU_DRAM_BYTES_PER_LAUNCH = {8192: 7795650304 + 570514944, 4096: 1103830000 + 134994688}


def _load_measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except OSError:
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        # `gpu_id` is what nvidia-smi's --id takes. nvidia-smi does not honour CUDA_VISIBLE_DEVICES, so
        # a CUDA ordinal may name another GPU of a shared box: pass the device's UUID ("GPU-...").
        self.gpu_index = gpu_id
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        chosen = [l for (t, l) in self.lines if t0 <= t <= t1] or [l for (_, l) in self.lines]
        for line in chosen:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons), "gpu": self.gpu_index}


def host_cores() -> int:
    """Cores this process may run on. Passed to the oracle explicitly: a launcher may export
    OMP_NUM_THREADS=1 for every rank (torch.distributed.run does), which would otherwise make the
    CPU baseline a single-thread figure."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def oracle_slab_rate(A, B, C, rows: int, threads: int = 0):
    """Times the oracle (as it stands) on the first `rows` rows of the problem; returns
    (TFLOP/s, seconds, threads used)."""
    import oracle
    oracle.build()
    a = A[:rows].numpy()
    c = C[:rows].clone().numpy()
    b = B.numpy()
    threads = threads if threads > 0 else host_cores()
    t0 = time.perf_counter()
    oracle.dgemm_oracle(a, b, c, threads)
    dt = time.perf_counter() - t0
    flop = 2.0 * rows * B.shape[0] * B.shape[1]
    return flop / dt / 1e12, dt, threads


def time_shape(dg, torch, M, N, K, lda=None, ldb=None, ldc=None, min_ms=40.0):
    """Mean CUDA-event time (ms) of back-to-back dgemm_f64 calls on one synthetic problem."""
    lda, ldb, ldc = lda or K, ldb or N, ldc or N
    A = torch.rand(M, lda, dtype=torch.float64, device="cuda") * 2 - 1
    B = torch.rand(K, ldb, dtype=torch.float64, device="cuda") * 2 - 1
    C = torch.rand(M, ldc, dtype=torch.float64, device="cuda") * 2 - 1
    pa, pb, pc = A.data_ptr(), B.data_ptr(), C.data_ptr()
    call = dg.load_library().dgemm_f64
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        call(M, N, K, pa, lda, pb, ldb, pc, ldc, None)
    e0.record()
    call(M, N, K, pa, lda, pb, ldb, pc, ldc, None)
    e1.record()
    torch.cuda.synchronize()
    reps = int(max(3, min(500, min_ms / max(e0.elapsed_time(e1), 1e-3))))
    best = float("inf")
    for _ in range(3):
        e0.record()
        for _ in range(reps):
            call(M, N, K, pa, lda, pb, ldb, pc, ldc, None)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / reps)
    return best


def single_call_latency_us(dg, torch, n, reps=30):
    """Median device time of ONE dgemm_f64 call on an idle GPU (synchronise, event, call, event), next
    to which the back-to-back figure of time_shape() is the throughput of a stream of calls."""
    A = torch.rand(n, n, dtype=torch.float64, device="cuda") * 2 - 1
    B = torch.rand(n, n, dtype=torch.float64, device="cuda") * 2 - 1
    C = torch.zeros(n, n, dtype=torch.float64, device="cuda")
    pa, pb, pc = A.data_ptr(), B.data_ptr(), C.data_ptr()
    call = dg.load_library().dgemm_f64
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    lat = []
    for i in range(reps + 3):
        torch.cuda.synchronize()
        e0.record()
        call(n, n, n, pa, n, pb, n, pc, n, None)
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            lat.append(e0.elapsed_time(e1) * 1e3)
    return statistics.median(lat)


def other_shapes(dg, torch, peak_tflops, hbm_gbs):
    """The square-size sweep (the metric's 'TFLOPS vs M=N=K' curve) and the ragged / rank-k shapes,
    each with its fraction of the FP64 peak and, for the low-intensity shapes, of the HBM roof."""
    sweep = []
    for n in range(128, 4096 + 1, 128):
        ms = time_shape(dg, torch, n, n, n)
        tf = 2.0 * n ** 3 / ms / 1e9
        row = {"n": n, "us": round(ms * 1e3, 1), "tflops": round(tf, 2), "frac_peak": round(tf / peak_tflops, 3)}
        if n <= 1024:  # latency-bound sizes: one isolated call beside the stream of calls
            row["single_call_us"] = round(single_call_latency_us(dg, torch, n), 1)
        sweep.append(row)
    shapes = []
    for (M, N, K, pad) in [(1000, 1537, 777, True), (2088, 2088, 2088, True), (4097, 31, 4099, True),
                           (2088, 2048, 2048, False), (16384, 16384, 64, False), (16384, 16384, 256, False),
                           # skinny shapes (narrow, short and half-width tiles), beyond the five configurations
                           (8192, 64, 8192, False), (32, 8192, 8192, False), (6514, 146, 4096, False)]:
        ld = (K + 3, N + 5, N + 7) if pad else (K, N, N)
        ms = time_shape(dg, torch, M, N, K, *ld)
        tf = 2.0 * M * N * K / ms / 1e9
        gbs = 8.0 * (M * K + K * N + 2 * M * N) / ms / 1e6
        shapes.append({"M": M, "N": N, "K": K, "ld": list(ld), "us": round(ms * 1e3, 1), "tflops": round(tf, 2),
                       "frac_peak": round(tf / peak_tflops, 3), "hbm_gbs": round(gbs), "frac_hbm": round(gbs / hbm_gbs, 3)})
    return sweep, shapes


def sgemm_section(dg, torch, sm_max_mhz, sizes=(2048, 4096, 8192)):
    """The paper's second workload (Section 2.13): C += A*B in binary32, here exact FP32 arithmetic
    on the FP32 pipe (packed FFMA). The path is bound by plain ALU arithmetic: peak = SMs x 128
    FMA/clk x 2 x clock. Timed like the FP64 headline, on resident operands."""
    peak = SM_COUNT_B200 * 128 * 2 * sm_max_mhz * 1e6 / 1e12
    out = {"dtype": "f32", "bound": "alu", "peak": peak, "unit": "TFLOP/s",
           "peak_source": "148 SMs x 128 FP32 FMA/clk x 2 x sm_max_mhz; a register-only packed-FMA loop sustains 85 % of it",
           "kernel": "sgemm_ffma_kernel<16, 2> (TMA staging, 256 x 128 x 32 tiles, 16 x 8 per thread, fma.rn.f32x2); 64-row and 64-column forms for the skinny shapes", "shapes": []}
    call = dg.load_library().sgemm_f32
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # the squares, then a short M (64-row tiles) and a narrow N (64-column tiles)
    skinny = [(32, 8192, 8192), (8192, 64, 8192)] if len(sizes) > 1 else []
    for shape in [(n, n, n) for n in sizes] + skinny:
        M, N, K = shape
        A = torch.rand(M, K, dtype=torch.float32, device="cuda") * 2 - 1
        B = torch.rand(K, N, dtype=torch.float32, device="cuda") * 2 - 1
        C = torch.zeros(M, N, dtype=torch.float32, device="cuda")
        pa, pb, pc = A.data_ptr(), B.data_ptr(), C.data_ptr()
        for _ in range(3):
            call(M, N, K, pa, K, pb, N, pc, N, None)
        torch.cuda.synchronize()
        reps = max(3, min(50, int(8192 ** 3 // (M * N * K)) * 3))
        best = float("inf")
        for _ in range(3):
            e0.record()
            for _ in range(reps):
                call(M, N, K, pa, K, pb, N, pc, N, None)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / reps)
        tf = 2.0 * M * N * K / best / 1e9
        entry = {"n": M} if M == N == K else {"M": M, "N": N, "K": K}
        entry.update({"us": round(best * 1e3, 1), "tflops": round(tf, 2), "frac": round(tf / peak, 3)})
        out["shapes"].append(entry)
        del A, B, C
    assert dg.sgemm_last_device_status() == 0
    return out


def ablation_ladder(dg, torch, peak_tflops, n=4096):
    """The paper walks from a naive nest to its best schedule step by step (Sections 2.3-2.9, Figure
    'journey'); this is the same walk on the GPU at M=N=K=n: each rung is a variant or test flag of
    the library. Returns a list of {rung, tflops, frac_peak}."""
    rungs = [
        ("naive nest, one thread per C element", dict(variant=dg.DGEMM_VARIANT_NAIVE, n=min(n, 2048))),
        ("+ tiles of A and B in shared memory, still one C element per thread (no register tile)",
         dict(variant=dg.DGEMM_VARIANT_SMEM, n=min(n, 2048))),
        ("+ 8x8 register tile per thread on plain FMAs (DFMA), 8-byte cp.async staging, mbarrier pipeline, 64x128 tile, 2 CTAs/SM",
         dict(variant=dg.DGEMM_VARIANT_GENERIC_DFMA, flags=16)),
        ("+ tensor-core micro-kernel (DMMA) in place of DFMA; same staging, 128x128 tile, 1 CTA/SM",
         dict(variant=dg.DGEMM_VARIANT_GENERIC, flags=4 | 16)),
        ("+ TMA staging (2-D copies, 9 per stage), no C prefetch", dict(variant=dg.DGEMM_VARIANT_TMA, flags=4 | 2 | 1)),
        ("+ one 3-D copy for B, C prefetch into L2", dict(variant=dg.DGEMM_VARIANT_TMA, flags=4)),
        ("32x32 warp tiles, 16 warps", dict(variant=dg.DGEMM_VARIANT_TMA, flags=4 | 8)),
        ("64x128 tiles, two CTAs per SM", dict(variant=dg.DGEMM_VARIANT_TMA)),
        ("producer warpgroup (setmaxnreg), software-pipelined consumers (default at this size)",
         dict(variant=dg.DGEMM_VARIANT_AUTO)),
    ]
    out = []
    for name, cfg in rungs:
        m = cfg.get("n", n)
        dg.dgemm_set_variant(cfg["variant"])
        dg.dgemm_set_test_flags(cfg.get("flags", 0))
        try:
            ms = time_shape(dg, torch, m, m, m)
        finally:
            dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
            dg.dgemm_set_test_flags(0)
        tf = 2.0 * m ** 3 / ms / 1e9
        out.append({"rung": name, "n": m, "tflops": round(tf, 2), "frac_peak": round(tf / peak_tflops, 3)})
    return out


def micro_kernel_swap(dg, torch, peak_tflops, n=4096):
    """The paper's 'outer MLIR, inner BLIS' experiment (Section 2.12) on the GPU: one macro-kernel (TMA
    staging, mbarrier pipeline, grouped raster, stream-K tail, epilogue; 64 x 128 tiles, two CTAs per
    SM) with two inner kernels, tensor-core MMAs and plain FMAs on the same 8 x 8 register tile per
    thread. Each is set against the ceiling of its own instruction, measured by a register-only loop."""
    _, fma_ceiling = dg.dgemm_fp64_fma_probe(300)
    fma_per_clk, _ = dg.dgemm_fp64_fma_probe(100)
    out = {"n": n, "macro_kernel": "dgemm_dmma_kernel<TMA, 64 x 128 x 16, 4 stages, 2 CTAs/SM>",
           "dfma_ceiling_tflops": round(fma_ceiling, 2), "dfma_fma_per_clk_sm": round(fma_per_clk, 1)}
    for key, variant, ceiling in (("dmma", dg.DGEMM_VARIANT_TMA, peak_tflops), ("dfma", dg.DGEMM_VARIANT_TMA_DFMA, fma_ceiling)):
        dg.dgemm_set_variant(variant)
        try:
            ms = time_shape(dg, torch, n, n, n)
        finally:
            dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        tf = 2.0 * n ** 3 / ms / 1e9
        out[key] = {"tflops": round(tf, 2), "frac_of_own_ceiling": round(tf / ceiling, 3), "frac_peak": round(tf / peak_tflops, 3)}
    return out


def run_reference(args):
    """The oracle on the host cores: each step is a bounded row slab of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from paper_2003_00532_b200 import workloads as wl
    n = args.size
    rows = min(args.ref_rows, n)
    prob = wl.make_problem(rows, n, n, 1)  # same distribution/seed; only `rows` rows of A and C are needed
    times = []
    cores = 0
    for step in range(args.warmup + args.steps):
        tf, dt, cores = oracle_slab_rate(prob.A, prob.B, prob.C, rows)
        if step >= args.warmup:
            times.append(dt)
    total = sum(times)
    flop = 2.0 * rows * n * n * len(times)
    value = flop / total / 1e12
    sample = f"{rows} of {n} rows of C per step (rows are independent and equal-cost), all {n} columns and k"
    line = {
        "impl": "reference", "metric": "dgemm_fp64_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"M=N=K={n} FP64 row-major, uniform [-1,1), seed 1", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2003_00532_b200 as dg
    from paper_2003_00532_b200 import replicas
    from paper_2003_00532_b200 import workloads as wl

    rank, local_rank, world = replicas.rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    distributed = world > 1
    if distributed:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return replicas.max_over_ranks(x, device="cuda")

    dg.load_library()
    if args.variant != dg.DGEMM_VARIANT_AUTO or args.flags:
        dg.dgemm_set_variant(args.variant)   # profiling aid: one rung of the ladder as the timed kernel
        dg.dgemm_set_test_flags(args.flags)
    n = args.size
    if args.shape:
        sm, sn, sk = (int(x) for x in args.shape.split(","))
        pad = dict(lda=sk + 3, ldb=sn + 5, ldc=sn + 7) if args.pad else {}  # the ragged configuration's leading dimensions
        prob = wl.make_problem(sm, sn, sk, 2 if args.pad else 3, pin=True, **pad)  # another shape (profiling aid)
    else:
        sm = sn = sk = n
        prob = wl.make_problem(n, n, n, 1, pin=True)  # seed 1: the large square configuration
    A_dev, B_dev, C_dev = prob.A_buf.cuda(), prob.B_buf.cuda(), prob.C_buf.cuda()
    A, B, C = A_dev[:, :sk], B_dev[:, :sn], C_dev[:, :sn]  # the logical matrices inside their (possibly padded) buffers
    flop = prob.flop
    stream = torch.cuda.current_stream()

    # ---- device-resident timing ------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        dg.dgemm_f64(A, B, C, stream=stream)
    barrier()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:  # noqa: BLE001 - an older torch without the uuid property
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    launches0 = dg.dgemm_launch_count()
    barrier()
    t_wall0 = time.time()
    events[0].record(stream)
    for i in range(args.steps):
        dg.dgemm_f64(A, B, C, stream=stream)
        events[i + 1].record(stream)
    barrier()
    t_wall1 = time.time()
    launches = dg.dgemm_launch_count() - launches0
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    status = dg.dgemm_last_device_status(stream)
    if status != 0:
        raise RuntimeError("device status: " + dg.dgemm_strerror(status))
    step_ms = [events[i].elapsed_time(events[i + 1]) for i in range(args.steps)]
    total_ms = max_over_ranks(events[0].elapsed_time(events[args.steps]))
    value = world * flop * args.steps / (total_ms * 1e-3) / 1e12
    kernel_ms = sum(step_ms) / len(step_ms)  # one kernel per step: launch duration on its stream

    # ---- end to end through the host entry point -----------------------------------------
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    dg.dgemm_f64_host(prob.A, prob.B, prob.C)  # warm-up (allocator pools, page locks)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        dg.dgemm_f64_host(prob.A, prob.B, prob.C)
    barrier()
    e2e_s = max_over_ranks(time.perf_counter() - t0)
    e2e_value = world * flop * e2e_steps / e2e_s / 1e12
    h2d = 8 * (sm * sk + sk * sn + sm * sn)
    d2h = 8 * sm * sn
    # what the host link of this machine gives a plain pinned copy (context for the end-to-end number,
    # which moves h2d + d2h bytes per step over it): one copy of A each way, outside the timed regions
    link = {}
    if rank == 0:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        A_dev.copy_(prob.A_buf, non_blocking=True)  # warm-up
        torch.cuda.synchronize()
        ev[0].record(stream)
        A_dev.copy_(prob.A_buf, non_blocking=True)
        ev[1].record(stream)
        prob.A_buf.copy_(A_dev, non_blocking=True)
        ev[2].record(stream)
        torch.cuda.synchronize()
        nbytes = A_dev.numel() * 8
        link = {"h2d_gbs": nbytes / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9,
                "d2h_gbs": nbytes / (ev[1].elapsed_time(ev[2]) * 1e-3) / 1e9}
        link["floor_ms_per_step"] = max(h2d / (link["h2d_gbs"] * 1e9), d2h / (link["d2h_gbs"] * 1e9)) * 1e3

    # the host entry point ran on streams of its own, which switched the library's scratch pool to its
    # multi-stream mode (an event per call); give the scratch back so that the single-stream timings
    # below run as a single-stream program does
    dg.dgemm_release_scratch()
    if args.variant != dg.DGEMM_VARIANT_AUTO or args.flags:
        dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
        dg.dgemm_set_test_flags(0)

    if rank != 0:
        if distributed:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel ---------------------------------------------------
    peaks = _load_measured_peaks()
    sm_max_mhz = float(peaks["sm_max_mhz"]) if peaks and "sm_max_mhz" in peaks else 1965.0
    peak_tflops = SM_COUNT_B200 * FMA_PER_CLK_SM * 2 * sm_max_mhz * 1e6 / 1e12
    # sustained issue rate: back-to-back register-only launches of 500 ms for --probe-ms in all (no
    # single multi-second kernel); the mean is the sustained figure, the first launch the burst one
    probe_runs = [dg.dgemm_fp64_peak_probe(500) for _ in range(max(1, args.probe_ms // 500))]
    probe_fma = statistics.mean(r[0] for r in probe_runs)
    probe_tflops = statistics.mean(r[1] for r in probe_runs)
    achieved = flop / (kernel_ms * 1e-3) / 1e12
    hbm_gbs = float(peaks["hbm_gbs"]) if peaks and "hbm_gbs" in peaks else 6650.0
    roofline = {
        "bound": "tensor", "achieved": achieved, "peak": peak_tflops, "unit": "TFLOP/s",
        "frac": achieved / peak_tflops, "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(n) if not args.shape else None,
        "kernel": "dgemm_dmma_ws_kernel<true> (TMA staging, 128 x 128 tiles, 8 consumer warps + producer warpgroup per SM)",
        "peak_source": (f"FP64 DMMA issue rate {FMA_PER_CLK_SM} FMA/clk/SM (measured by the register-only probe) x "
                        f"{SM_COUNT_B200} SMs x 2 x sm_max_mhz {sm_max_mhz:.0f} "
                        f"({'MEASURED_PEAKS.json' if peaks else 'fallback 1965'}); MEASURED_PEAKS has no FP64 entry"),
        "probe_fma_per_clk_sm": probe_fma, "probe_sustained_tflops": probe_tflops,
        "probe_seconds": 0.5 * len(probe_runs), "probe_burst_tflops": probe_runs[0][1],
        "probe_min_tflops": min(r[1] for r in probe_runs),
        "frac_of_probe_sustained": achieved / probe_tflops if probe_tflops > 0 else None,
        "algorithmic_flop_per_launch": flop,
        "algorithmic_bytes_per_launch": prob.min_bytes,
        "hbm_time_floor_ms": prob.min_bytes / (hbm_gbs * 1e9) * 1e3,
    }

    # ---- CPU baseline: the oracle as it stands, on a bounded row slab -------------------------
    cpu_rows = min(args.cpu_rows, sm)
    tf_cpu, dt_cpu, cores = oracle_slab_rate(prob.A, prob.B, prob.C, cpu_rows)
    cpu_baseline = {"value": tf_cpu, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                    "sample": f"{cpu_rows} of {sm} rows of C (rows are independent and equal-cost), "
                              f"{dt_cpu:.1f} s"}

    line = {
        "metric": "dgemm_fp64_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": (f"M=N=K={n} FP64 row-major C += A*B, A,B,C uniform [-1,1), seed 1" if not args.shape else
                                f"M,N,K={args.shape} FP64 row-major C += A*B, uniform [-1,1), seed 3"),
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "l2": "operands (1.6 GB at 8192) exceed the 126 MB L2; no flush between steps",
                   "pct_of_fp64_peak": 100.0 * value / world / peak_tflops},
        "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
                "api": "dgemm_f64_host (pinned host buffers)", "host_link": link},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if not args.no_sweep:
        line["sweep"], line["other_shapes"] = other_shapes(dg, torch, peak_tflops, hbm_gbs)
        line["ablation"] = ablation_ladder(dg, torch, peak_tflops)
        line["micro_kernel_swap"] = micro_kernel_swap(dg, torch, peak_tflops)
        line["sgemm"] = sgemm_section(dg, torch, sm_max_mhz)
    print(json.dumps(line), flush=True)
    if distributed:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--size", type=int, default=8192, help="M=N=K of the square workload")
    ap.add_argument("--ref-rows", type=int, default=128, help="rows of C per step of the reference arm")
    ap.add_argument("--cpu-rows", type=int, default=3072, help="rows of C in the cpu_baseline sample")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--shape", type=str, default="", help="M,N,K of another (non-square) workload; profiling aid")
    ap.add_argument("--pad", action="store_true", help="with --shape: padded leading dimensions lda=K+3, ldb=N+5, ldc=N+7, seed 2")
    ap.add_argument("--no-sweep", action="store_true", help="skip the size sweep and the ragged / rank-k shapes")
    ap.add_argument("--variant", type=int, default=-1, help="profiling aid: force a DGEMM_VARIANT_* for the timed calls")
    ap.add_argument("--flags", type=int, default=0, help="profiling aid: DGEMM_TEST_* flags for the timed calls")
    ap.add_argument("--probe-ms", type=int, default=4000,
                    help="total length of the sustained FP64 issue-rate probe (run as launches of 500 ms)")
    ap.add_argument("--sgemm-size", type=int, default=0,
                    help="profiling aid: time only sgemm_f32 at M=N=K of this size, print its section and exit")
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be >= 1")
    if args.sgemm_size:
        import torch
        import paper_2003_00532_b200 as dg
        torch.cuda.set_device(0)
        print(json.dumps(sgemm_section(dg, torch, 1965.0, sizes=(args.sgemm_size,))))
        return 0
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
