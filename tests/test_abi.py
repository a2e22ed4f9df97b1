"""The C-ABI library loads and exports every symbol declared in include/dgemm.h (no GPU needed),
and the oracle library exports what its header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared(header, pattern):
    text = open(header).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return re.findall(pattern, text)


@pytest.fixture(scope="module")
def lib():
    from paper_2003_00532_b200 import build as _build
    import paper_2003_00532_b200 as dg
    _build.build()
    return dg.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = _declared(os.path.join(ROOT, "include", "dgemm.h"), r"DGEMM_API\s+[\w\s\*]+?\b(dgemm_\w+)\s*\(")
    assert {"dgemm_f64", "dgemm_f64_ex", "dgemm_f64_host", "dgemm_f64_static_ws", "dgemm_strerror", "dgemm_version",
            "dgemm_set_variant", "dgemm_set_split_k", "dgemm_set_test_flags", "dgemm_last_device_status", "dgemm_launch_count",
            "dgemm_fp64_peak_probe", "dgemm_selftest_wait_timeout", "dgemm_plan", "dgemm_release_scratch"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in dgemm.h but not exported by libdgemm.so"
    names32 = _declared(os.path.join(ROOT, "include", "sgemm.h"), r"DGEMM_API\s+[\w\s\*]+?\b(sgemm_\w+)\s*\(")
    assert {"sgemm_f32", "sgemm_last_device_status"} <= set(names32)
    for n in names32:
        assert hasattr(lib, n), f"{n} is declared in sgemm.h but not exported by libdgemm.so"


def test_header_is_plain_c():
    import subprocess
    src = '#include "dgemm.h"\n#include "sgemm.h"\nint main(void){return DGEMM_OK + DGEMM_VARIANT_COUNT - 3;}\n'
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), "-x", "c", "-",
                    "-fsyntax-only"], input=src.encode(), check=True)


def test_status_codes_match_binding(lib):
    import paper_2003_00532_b200.binding as b
    text = open(os.path.join(ROOT, "include", "dgemm.h")).read()
    for name, val in re.findall(r"(DGEMM_(?:OK|ERR_\w+|VARIANT_\w+))\s*=\s*(-?\d+)", text):
        if name == "DGEMM_VARIANT_COUNT":
            continue
        assert getattr(b, name) == int(val), name
    msgs = {b.dgemm_strerror(c) for c in range(0, -11, -1)}
    assert len(msgs) == 11 and "unknown status" not in msgs
    assert b.dgemm_strerror(-99) == "unknown status"
    assert b.dgemm_version() >= 100


def test_oracle_library_exports(oracle):
    names = _declared(os.path.join(ROOT, "oracle", "dgemm_oracle.h"), r"\b(dgemm_oracle_\w+)\s*\(")
    lib = ctypes.CDLL(oracle.build())
    for n in set(names):
        assert hasattr(lib, n)


def test_product_and_oracle_share_no_code():
    """The oracle never imports the product and the product never imports the oracle."""
    for folder, banned in (("oracle", "paper_2003_00532_b200"), ("paper_2003_00532_b200", "oracle")):
        for dirpath, _, files in os.walk(os.path.join(ROOT, folder)):
            for f in files:
                if f.endswith((".py", ".c", ".h", ".cu", ".cuh")):
                    text = open(os.path.join(dirpath, f)).read()
                    assert not re.search(rf"^\s*(from|import)\s+{banned}\b", text, flags=re.M), (dirpath, f)
                    assert f'#include "../{banned}' not in text and f"{banned}/" not in text.replace(
                        "paper_2003_00532_b200.build", ""), (dirpath, f)
