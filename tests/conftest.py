import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); deselect with -m 'not gpu'")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle package, with its C library compiled."""
    import oracle as _oracle
    _oracle.build()
    return _oracle


# Largest observed error / stated-bound ratio per benchmark configuration, collected by the parity
# tests. With DGEMM_PARITY_REPORT=<path> in the environment the table is written there as JSON at
# the end of the session (documentation of the margin; the assertions themselves are in the tests).
_PARITY_RATIOS = {}


def record_ratio(name: str, ratio: float) -> None:
    _PARITY_RATIOS[name] = max(ratio, _PARITY_RATIOS.get(name, 0.0))


def pytest_sessionfinish(session, exitstatus):
    path = os.environ.get("DGEMM_PARITY_REPORT")
    if path and _PARITY_RATIOS:
        import json
        with open(path, "w") as f:
            json.dump(_PARITY_RATIOS, f, indent=1, sort_keys=True)
