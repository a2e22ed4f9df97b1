"""Builds ``libdgemm.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import shlex
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdgemm.so")
SOURCES = [os.path.join(CSRC, "dgemm_api.cu"), os.path.join(CSRC, "sgemm_api.cu")]
# every source, header and public header: an edit to any of them makes the built library stale
DEPS = sorted(glob.glob(os.path.join(CSRC, "*.cu")) + glob.glob(os.path.join(CSRC, "*.cuh")) +
              glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(os.path.dirname(HERE), "include", "*.h")))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-cudart", "static",
]


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in DEPS)


# What ptxas must report for the kernels whose speed hangs on their register allocation: (substring
# of the mangled name, registers per thread at launch, most bytes of spill stores tolerated). The
# warp-specialised kernels redistribute a pool of threads x registers with setmaxnreg, so another
# launch count changes the consumers' budget; the 8192^3 figure was measured with exactly these.
PTXAS_EXPECT = [
    ("dgemm_dmma_ws_kernelILb1ELi128ELb0ELb0EE", 168, 128),
    ("dgemm_dmma_ws_kernelILb1ELi64ELb0ELb0EE", 128, 128),
    ("dgemm_dmma_kernelILb1ELi64ELi64ELi128ELi0ELb0ELb0EE", 255, 64),
]


def check_ptxas(log: str) -> None:
    """Raises if the `-Xptxas -v` output in `log` departs from PTXAS_EXPECT (a toolchain that allocates
    registers differently would silently change the measured speed)."""
    import re
    found = {}
    current = None
    spill = 0
    for line in log.splitlines():
        m = re.search(r"Compiling entry function '([^']+)'", line)
        if m:
            current, spill = m.group(1), 0
            continue
        m = re.search(r"(\d+) bytes spill stores", line)
        if m and current:
            spill = int(m.group(1))
        m = re.search(r"Used (\d+) registers", line)
        if m and current:
            found[current] = (int(m.group(1)), spill)
            current = None
    problems = []
    for key, regs, max_spill in PTXAS_EXPECT:
        hits = [(name, v) for name, v in found.items() if key in name]
        if not hits:
            problems.append(f"{key}: not found in the ptxas output")
        for name, (r, sp) in hits:
            if r != regs or sp > max_spill:
                problems.append(f"{name}: {r} registers, {sp} bytes of spill stores; expected {regs} and at most {max_spill}")
    if problems:
        raise RuntimeError("ptxas resource usage changed:\n  " + "\n  ".join(problems))


def build(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path. With `check`
    the compile reports resource usage and fails if the hot kernels' registers or spills changed."""
    if force or is_stale():
        tmp = LIB + ".tmp.%d" % os.getpid()
        extra = shlex.split(os.environ.get("DGEMM_NVCC_FLAGS", ""))  # e.g. -D switches for experiments
        cmd = [nvcc_path(), *NVCC_FLAGS, *extra, *(["-Xptxas", "-v"] if (verbose or check) else []), "-o", tmp, *SOURCES]
        res = subprocess.run(cmd, cwd=CSRC, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed building libdgemm.so")
        if check and not extra:
            check_ptxas(res.stdout + res.stderr)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
