import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def read_golden(name):
    """Parse a tests/golden/*.txt fixture: '#' comments, 'key = v1 v2 ...' lines (repeatable)."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=", 1)
            out.setdefault(k.strip(), []).append([float(x) for x in v.split()])
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
