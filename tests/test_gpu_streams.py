"""Calls in flight on several streams at once. Needs a B200.

The library owns scratch memory (partial tiles of split K, packed copies of operands TMA cannot
address). Each call leases its own share, so calls on different streams, from one host thread or
several, must not disturb each other. Every case here uses integer-valued data and is compared bit
for bit with the CPU oracle: a partial tile or a packed operand overwritten by the other stream's
call cannot go unnoticed.
"""
import threading

import numpy as np
import pytest
import torch

import paper_2003_00532_b200 as dg
from paper_2003_00532_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _oracle_result(oracle, prob):
    want = prob.C.clone().contiguous().numpy()
    oracle.dgemm_oracle(np.ascontiguousarray(prob.A.numpy()), np.ascontiguousarray(prob.B.numpy()), want)
    return want


class _Job:
    """One problem with device copies, a stream of its own and its expected result."""

    def __init__(self, oracle, M, N, K, seed, ld=None):
        lda, ldb, ldc = ld if ld else (K, N, N)
        self.prob = wl.make_problem(M, N, K, seed=seed, lda=lda, ldb=ldb, ldc=ldc, integer=True)
        self.want = _oracle_result(oracle, self.prob)
        self.A, self.B = self.prob.A_buf.cuda(), self.prob.B_buf.cuda()
        self.C0 = self.prob.C_buf.cuda()
        self.C = self.C0.clone()
        self.stream = torch.cuda.Stream()

    def reset(self):
        self.C.copy_(self.C0)

    def launch(self):
        p = self.prob
        dg.dgemm_f64(self.A[:, :p.K], self.B[:, :p.N], self.C[:, :p.N], stream=self.stream)

    def check(self, what):
        out = self.C.cpu()
        assert wl.c_padding_intact(out, self.prob.N), what
        got = np.ascontiguousarray(out[:, :self.prob.N].numpy())
        assert got.tobytes() == self.want.tobytes(), what


def test_two_streams_that_both_use_the_workspace(oracle):
    """(1000, 1537, 777) splits the K of its last wave through the workspace; 2088^3 with odd leading
    dimensions is packed into scratch first and also has a split last wave. Twenty rounds, both
    in flight at the same time."""
    jobs = [_Job(oracle, 1000, 1537, 777, seed=2, ld=(780, 1542, 1544)),
            _Job(oracle, 2088, 2088, 2088, seed=3, ld=(2091, 2093, 2095))]
    torch.cuda.synchronize()
    for rnd in range(20):
        for j in jobs:
            j.reset()
        torch.cuda.synchronize()
        for j in (jobs if rnd % 2 == 0 else jobs[::-1]):
            j.launch()
        assert all(dg.dgemm_last_device_status(j.stream) == dg.DGEMM_OK for j in jobs)
        for j in jobs:
            j.check(f"round {rnd}")


def test_more_streams_than_leases(oracle):
    """Six streams, each with a small problem whose K is cut through the workspace (forced split),
    several calls per stream without any synchronisation in between: more concurrent users than the
    pool has leases, so late comers wait for the least recently used lease's last user."""
    shapes = [(300, 200, 1000), (260, 300, 777), (129, 257, 515), (200, 150, 1000), (384, 128, 640), (100, 500, 333)]
    jobs = [_Job(oracle, M, N, K, seed=40 + i) for i, (M, N, K) in enumerate(shapes)]
    dg.dgemm_set_split_k(4)
    try:
        torch.cuda.synchronize()
        for rnd in range(10):
            for j in jobs:
                j.reset()
            torch.cuda.synchronize()
            for j in jobs:
                j.launch()
            torch.cuda.synchronize()
            for j in jobs:
                j.check(f"round {rnd}")
    finally:
        dg.dgemm_set_split_k(0)
    assert dg.dgemm_last_device_status() == dg.DGEMM_OK


def test_two_host_threads_two_streams(oracle):
    """Two host threads, each calling on a stream of its own, at the same time."""
    jobs = [_Job(oracle, 1000, 1537, 777, seed=5, ld=(780, 1542, 1544)),
            _Job(oracle, 700, 650, 1200, seed=6, ld=(1203, 655, 657))]
    torch.cuda.synchronize()
    errors = []

    def worker(job):
        try:
            torch.cuda.set_device(0)
            for rnd in range(15):
                with torch.cuda.stream(job.stream):
                    job.reset()
                job.launch()
                job.stream.synchronize()
                job.check(f"round {rnd}")
        except Exception as exc:  # noqa: BLE001 - reported to the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert dg.dgemm_last_device_status() == dg.DGEMM_OK


def test_back_to_one_stream_after_release(oracle):
    """dgemm_release_scratch gives every lease back; afterwards the library starts over (one lease,
    no events while a single stream is in use) and results are unchanged."""
    job = _Job(oracle, 1000, 1537, 777, seed=7, ld=(780, 1542, 1544))
    assert dg.dgemm_release_scratch() == dg.DGEMM_OK
    for _ in range(3):
        job.reset()
        job.launch()
        assert dg.dgemm_last_device_status(job.stream) == dg.DGEMM_OK
        job.check("after release")
