import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (B200)")


def read_golden(name):
    """Parse a tests/golden/*.txt fixture: '#' comments, 'key v v v' lines -> dict of lists
    (repeated keys accumulate a list of lists)."""
    path = os.path.join(ROOT, "tests", "golden", name)
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            parts = line.split()
            key, vals = parts[0], parts[1:]
            out.setdefault(key, []).append(vals)
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
