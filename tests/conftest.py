import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")
    # The tests call the C-ABI library; build it in-tree (nvcc cross-compiles without a GPU) when a fresh
    # checkout has not done so yet.
    from paper_2609_32704_b200.build import LIB_PATH, build_library
    if not os.path.exists(LIB_PATH):
        build_library()


def read_golden(name):
    rows = []
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(x) for x in line.split()])
    return rows


@pytest.fixture(scope="session")
def golden():
    return read_golden
