import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def read_golden(name):
    """Parse a golden fixture into {key: [tokens]} (first token of a line is the key);
    lines that repeat a key are collected as a list of rows under that key."""
    rows = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            tok = line.split()
            rows.setdefault(tok[0], []).append(tok[1:])
    return rows


@pytest.fixture(scope="session")
def golden():
    return read_golden
