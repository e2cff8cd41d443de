import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


def read_golden(path):
    """A golden file is text: '#' lines are comments (the citation), the rest whitespace-separated numbers per line."""
    rows = []
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                rows.append([float(x) for x in line.split()])
    return rows


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Both shared libraries are built in-tree before any test runs (nvcc cross-compiles without a GPU)."""
    from paper_2403_11805_b200 import build as gpu_build
    from oracle import build as oracle_build
    oracle_build.build()
    gpu_build.build()
