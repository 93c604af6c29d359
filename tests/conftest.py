import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def golden(name):
    """Parse a tests/golden/*.txt fixture: '#' lines are citations, the rest 'key value...' rows."""
    rows = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            rows[parts[0]] = [float(v) for v in parts[1:]]
    return rows


@pytest.fixture(scope="session")
def oracle():
    from oracle import oracle_a48
    oracle_a48.build()
    return oracle_a48


@pytest.fixture(scope="session")
def a48():
    """The ctypes binding over the CUDA library, built in-tree on first use."""
    from paper_2411_04965_b200 import binding, build
    build.build()
    binding.lib()
    return binding


@pytest.fixture(scope="session")
def cuda_dev():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("a test marked gpu ran without a CUDA device")
    return torch.device("cuda:0")
