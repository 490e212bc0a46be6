import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu")


def read_golden(name):
    """Parse a `key = value  # citation` text fixture into {key: (value_string, citation)}."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            body, _, cite = line.partition("#")
            key, _, val = body.partition("=")
            out[key.strip()] = (val.strip(), cite.strip())
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
