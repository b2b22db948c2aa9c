import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def read_golden(name):
    """Parse a golden text fixture: '#' comments, then 'key: v v v' lines -> dict of
    lists of strings."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = line.split(":", 1)
            out.setdefault(k.strip(), []).append(v.split())
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
