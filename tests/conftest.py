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


def pytest_sessionfinish(session, exitstatus):
    """When COWA_PARITY_ERRORS names a file, writes there the largest errors the parity tests measured at the
    benchmark configurations (max-abs, mean of the mean-abs errors, largest reference magnitude): the source of
    the error table in the design notes."""
    path = os.environ.get("COWA_PARITY_ERRORS")
    mod = sys.modules.get("test_gpu_parity") or sys.modules.get("tests.test_gpu_parity")
    measured = getattr(mod, "MEASURED", None) if mod else None
    if not path or not measured:
        return
    import json
    rows = [{"config": c, "tensor": t, "max_abs": v[0], "mean_abs": v[1] / max(v[2], 1), "checks": v[2],
             "max_abs_reference": v[3]} for (c, t), v in sorted(measured.items())]
    with open(path, "w") as f_:
        json.dump(rows, f_, indent=1)
