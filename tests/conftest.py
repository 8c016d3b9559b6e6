import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a library)")


def read_golden(name):
    """Parse a `key = value` fixture under tests/golden/ (comment lines start with #)."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, value = [s.strip() for s in line.split("=", 1)]
            out[key] = float(value) if "." in value else int(value)
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
