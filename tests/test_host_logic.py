"""Host-side logic that needs no GPU: argument validation order of the C ABI, the binding's
marshalling, the workload generators and the replica aggregation over gloo (world size 2)."""
import os

import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2003_00532_b200 import build as _build
    _build.build()


def test_validation_needs_no_device():
    f = dg.dgemm_f64_raw
    a, b, c = 4096, 8192, 16384  # never dereferenced: every call below fails validation first
    assert f(-1, 1, 1, a, 1, b, 1, c, 1, check=False) == -1
    assert f(1, -1, 1, a, 1, b, 1, c, 1, check=False) == -1
    assert f(1, 1, -1, a, 1, b, 1, c, 1, check=False) == -1
    assert f(2 ** 31, 1, 1, a, 1, b, 1, c, 1, check=False) == -1
    assert f(0, 5, 5, None, 5, None, 5, None, 5) == 0          # M = 0: nothing inspected
    assert f(5, 0, 5, None, 5, None, 1, None, 1) == 0          # N = 0
    assert f(2, 2, 2, a, 1, b, 2, c, 2, check=False) == -2     # lda < K
    assert f(2, 2, 2, a, 2, b, 1, c, 2, check=False) == -2     # ldb < N
    assert f(2, 2, 2, a, 2, b, 2, c, 1, check=False) == -2     # ldc < N
    assert f(2, 2, 0, a, 0, b, 2, c, 2, check=False) == -2     # lda >= 1 even when K = 0
    assert f(2, 2, 0, None, 1, None, 2, None, 2) == 0          # K = 0: C untouched, no pointers needed
    assert f(2, 2, 2, None, 2, b, 2, c, 2, check=False) == -3
    assert f(2, 2, 2, a, 2, b, 2, None, 2, check=False) == -3
    assert f(2, 2, 2, a + 4, 2, b, 2, c, 2, check=False) == -4
    assert f(2, 2, 2, a, 2, b, 2, a + 8, 2, check=False) == -5  # C inside A
    assert f(2, 2, 2, a, 2, b, 2, b - 8, 2, check=False) == -5  # C's tail reaches B
    with pytest.raises(dg.DgemmError) as e:
        f(2, 2, 2, a, 2, b, 2, b, 2)
    assert e.value.status == -5 and "overlaps" in str(e.value)
    g = dg.load_library().dgemm_f64_static_ws
    assert g(2, 2, 2, a, 2, b, 2, c, 2, -1, None) == -9
    assert g(-2, 2, 2, a, 2, b, 2, c, 2, 0, None) == -1
    h = dg.load_library().dgemm_f64_host
    assert h(2, 2, 2, a, 1, b, 2, c, 2) == -2


def test_sgemm_validation_needs_no_device():
    f = dg.load_library().sgemm_f32
    a, b, c = 4096, 8192, 16384  # never dereferenced: every call below fails validation first
    assert f(-1, 1, 1, a, 1, b, 1, c, 1, None) == -1
    assert f(2 ** 31, 1, 1, a, 1, b, 1, c, 1, None) == -1
    assert f(0, 5, 5, None, 5, None, 5, None, 5, None) == 0          # M = 0: nothing inspected
    assert f(5, 0, 5, None, 5, None, 1, None, 1, None) == 0          # N = 0
    assert f(2, 2, 2, a, 1, b, 2, c, 2, None) == -2                  # lda < K
    assert f(2, 2, 2, a, 2, b, 1, c, 2, None) == -2                  # ldb < N
    assert f(2, 2, 2, a, 2, b, 2, c, 1, None) == -2                  # ldc < N
    assert f(2, 2, 0, None, 1, None, 2, None, 2, None) == 0          # K = 0: C untouched
    assert f(2, 2, 2, None, 2, b, 2, c, 2, None) == -3
    assert f(2, 2, 2, a + 2, 2, b, 2, c, 2, None) == -4              # 4-byte alignment
    assert f(2, 2, 2, a + 4, 2, b, 2, a + 8, 2, None) == -5          # C inside A (A spans 16 bytes from a + 4)
    assert f(2, 2, 2, a, 2, b, 2, b - 4, 2, None) == -5              # C's tail reaches B


def test_general_form_validation_needs_no_device():
    x = dg.load_library().dgemm_f64_ex
    a, b, c = 4096, 8192, 16384
    N_, T_ = dg.DGEMM_OP_N, dg.DGEMM_OP_T
    assert x(2, N_, 2, 2, 2, 1.0, a, 2, b, 2, 1.0, c, 2, None) == -1      # unknown op code
    assert x(N_, -1, 2, 2, 2, 1.0, a, 2, b, 2, 1.0, c, 2, None) == -1
    # leading dimensions follow the STORED shapes: A^T is K x M (lda >= M), B^T is N x K (ldb >= K)
    assert x(N_, N_, 5, 3, 2, 1.0, a, 2, b, 3, 1.0, c, 2, None) == -2      # ldc < N
    assert x(T_, N_, 5, 3, 2, 1.0, a, 4, b, 3, 1.0, c, 3, None) == -2      # lda = 4 < M = 5
    assert x(N_, T_, 5, 3, 2, 1.0, a, 2, b, 1, 1.0, c, 3, None) == -2      # ldb = 1 < K = 2
    assert x(T_, T_, 5, 3, 2, 1.0, a, 5, b, 2, 1.0, None, 3, None) == -3
    # aliasing uses the stored extents: A^T (2 x 5, lda 5) spans 80 bytes
    assert x(T_, N_, 5, 3, 2, 1.0, a, 5, b, 3, 1.0, a + 72, 3, None) == -5
    assert x(N_, N_, 5, 3, 2, 1.0, a, 2, b, 3, 1.0, a + 72, 3, None) == -5  # A (5 x 2, lda 2) spans 80 bytes too
    assert x(N_, N_, 0, 3, 2, 0.0, None, 2, None, 3, 0.0, None, 3, None) == 0  # M = 0
    # nothing to do at all: beta = 1 and no product
    assert x(N_, N_, 2, 2, 0, 1.0, None, 1, None, 2, 1.0, None, 2, None) == 0
    assert x(N_, N_, 2, 2, 2, 0.0, None, 2, None, 2, 1.0, None, 2, None) == 0
    # C = beta * C needs C (and only C) when there is no product
    assert x(N_, N_, 2, 2, 2, 0.0, None, 2, None, 2, 0.5, None, 2, None) == -3
    assert x(N_, N_, 2, 2, 0, 1.0, None, 1, None, 2, 0.0, c + 4, 2, None) == -4


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a box without a GPU")
def test_valid_call_without_gpu_fails_loudly():
    A = torch.zeros(4, 4, dtype=torch.float64)
    rc = dg.dgemm_f64_raw(4, 4, 4, A.data_ptr(), 4, A.data_ptr(), 4, A.data_ptr() + 4096, 4, check=False)
    assert rc == -6  # no device: an error, never a CPU fallback
    with pytest.raises(dg.DgemmError):
        dg.dgemm_fp64_peak_probe(1)
    with pytest.raises(dg.DgemmError):
        dg.dgemm_release_scratch()


def test_variant_and_split_setters():
    assert dg.dgemm_set_variant(dg.DGEMM_VARIANT_GENERIC) == 0
    assert dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO) == 0
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_variant(dg.binding.DGEMM_VARIANT_TMA_WS_BULK + 1)
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_variant(-2)
    assert dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA_WS) == 0 and dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO) == 0
    assert dg.dgemm_set_variant(dg.DGEMM_VARIANT_TMA_CLUSTER) == 0 and dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO) == 0
    assert dg.dgemm_set_variant(dg.DGEMM_VARIANT_GENERIC_CLUSTER) == 0 and dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO) == 0
    assert dg.dgemm_set_test_flags(3) == 0 and dg.dgemm_set_test_flags(0) == 0
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_test_flags(512)
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_test_flags(64)   # not a flag
    assert dg.dgemm_set_split_k(4) == 0 and dg.dgemm_set_split_k(0) == 0
    with pytest.raises(dg.DgemmError):
        dg.dgemm_set_split_k(-1)
    assert dg.dgemm_launch_count() >= 0


def test_binding_marshalling_rejects_bad_tensors():
    A = torch.zeros(4, 4, dtype=torch.float64)
    with pytest.raises(ValueError):
        dg.dgemm_f64(A, A, A)                      # host tensors on the device entry point
    with pytest.raises(TypeError):
        dg.dgemm_f64_host(A.float(), A, A)
    with pytest.raises(ValueError):
        dg.dgemm_f64_host(A.t(), A, A.clone())     # column-major view
    with pytest.raises(ValueError):
        dg.dgemm_f64_host(torch.zeros(4, 3, dtype=torch.float64), A, A.clone())
    from paper_2003_00532_b200.binding import _matrix_args
    buf = torch.zeros(5, 10, dtype=torch.float64)
    assert _matrix_args(buf[:, :7], "x", False)[1:] == (5, 7, 10)
    assert _matrix_args(buf[:1, :7], "x", False)[1:] == (1, 7, 10)
    assert _matrix_args(torch.zeros(0, 7, dtype=torch.float64), "x", False)[1:] == (0, 7, 7)


def test_workload_generators():
    p = wl.make_problem(5, 7, 3, seed=2, lda=6, ldb=12, ldc=14)
    q = wl.make_problem(5, 7, 3, seed=2, lda=6, ldb=12, ldc=14)
    assert torch.equal(p.A, q.A) and torch.equal(p.B, q.B) and torch.equal(p.C, q.C)
    assert p.A.min() >= -1 and p.A.max() < 1
    assert torch.isnan(p.A_buf[:, 3:]).all() and torch.isnan(p.B_buf[:, 7:]).all()
    assert wl.c_padding_intact(p.C_buf, 7)
    p.C_buf[2, 9] = 0.0
    assert not wl.c_padding_intact(p.C_buf, 7)
    # draw order A, B, C from one generator: the dense problem shares A with the padded one
    d = wl.make_problem(5, 7, 3, seed=2)
    assert torch.equal(d.A, p.A) and torch.equal(d.B, p.B) and torch.equal(d.C, p.C)
    i = wl.make_problem(50, 40, 30, seed=0, integer=True, c_zero=True)
    assert set(i.A.unique().tolist()) <= set(range(-4, 5)) and i.A.min() == -4 and i.A.max() == 4
    assert (i.C == 0).all() and not torch.signbit(i.C).any()
    assert wl.config2_sizes()[0] == 128 and wl.config2_sizes()[-1] == 4096 and len(wl.config2_sizes()) == 32
    p4 = wl.config4(0)
    assert (p4.M, p4.N, p4.K, p4.lda, p4.ldb, p4.ldc) == (1000, 1537, 777, 780, 1542, 1544)
    ii, jj = wl.sample_indices(1000, 1537, 256, seed=1)
    assert len(ii) == 256 and ii.max() < 1000 and jj.max() < 1537 and (0 in ii.tolist()) and (999 in ii.tolist())
    assert p4.flop == 2.0 * 1000 * 1537 * 777
    assert p4.min_bytes == 8.0 * (1000 * 777 + 777 * 1537 + 2 * 1000 * 1537)


def _replica_worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2003_00532_b200.replicas import aggregate_rate, max_over_ranks
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local = 2.0 if rank == 0 else 5.0     # rank 1 is the slow replica
        dist.barrier()
        q.put((rank, max_over_ranks(local), aggregate_rate(100.0, local, world)))
    finally:
        dist.destroy_process_group()


def test_replicas_gloo_world_size_2():
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_replica_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, rate in out:
        assert mx == 5.0                      # every rank sees the slowest time
        assert rate == 2 * 100.0 / 5.0        # all replicas' units over the slowest time


def test_replicas_without_process_group():
    from paper_2003_00532_b200.replicas import aggregate_rate, rank_info
    assert aggregate_rate(10.0, 2.0, 1) == 5.0
    assert rank_info({"RANK": "3", "LOCAL_RANK": "1", "WORLD_SIZE": "8"}) == (3, 1, 8)
    assert rank_info({}) == (0, 0, 1)


def test_every_included_file_is_a_build_dependency():
    """An edit to any file the library is compiled from must make the built library stale."""
    import re
    from paper_2003_00532_b200 import build as b
    deps = {os.path.basename(d) for d in b.DEPS}
    for src in os.listdir(b.CSRC):
        if not src.endswith((".cu", ".cuh", ".h")):
            continue
        assert src in deps
        for inc in re.findall(r'#include\s+"([^"]+)"', open(os.path.join(b.CSRC, src)).read()):
            assert os.path.basename(inc) in deps, f"{src} includes {inc}, which build.DEPS does not list"


def test_ptxas_check_catches_a_changed_register_count():
    from paper_2003_00532_b200 import build as b
    good = "".join(
        f"ptxas info    : Compiling entry function '_ZN5dgemm{key}Ev' for 'sm_100a'\n"
        f"    8 bytes stack frame, {spill} bytes spill stores, 8 bytes spill loads\n"
        f"ptxas info    : Used {regs} registers, used 2 barriers\n" for key, regs, spill in b.PTXAS_EXPECT)
    b.check_ptxas(good)
    with pytest.raises(RuntimeError):
        b.check_ptxas(good.replace("Used 168 registers", "Used 160 registers"))
    with pytest.raises(RuntimeError):
        b.check_ptxas(good.replace("128 bytes spill stores", "4000 bytes spill stores", 1))
    with pytest.raises(RuntimeError):
        b.check_ptxas("")


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` times the CPU oracle (no GPU involved) and prints one JSON line
    with the same metric, unit and configuration keys as the library's own arm."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "dgemm_fp64_tflops" and line["unit"] == "TFLOP/s"
    assert line["higher_is_better"] is True and line["steps"] == 1 and line["warmup"] == 1 and line["n_gpus"] == 1
    assert line["value"] > 0 and line["ms_per_step"] > 0 and line["vs_baseline"] is None
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["cpu_baseline"]["cores"] >= 1 and line["cpu_baseline"]["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": line["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in line["config"]
