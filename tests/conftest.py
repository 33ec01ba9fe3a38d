import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def read_golden(name):
    """Rows of a whitespace-separated golden file, comments dropped."""
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if line:
                rows.append(line.split())
    return rows


@pytest.fixture(scope="session")
def lib():
    """The built C-ABI library (built on demand; needs nvcc, not a GPU)."""
    from paper_2403_20041_b200 import build as _build

    _build.build()
    from paper_2403_20041_b200 import binding

    return binding


@pytest.fixture
def tuning(lib):
    """Sets launch-heuristic overrides through tl_e0m4_tuning_set and restores all of them afterwards."""
    yield lib.tl_e0m4_tuning_set
    lib.tl_e0m4_tuning_set(None)
