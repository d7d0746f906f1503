import os
import sys

import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def read_golden(name):
    """Parse a 'key v1 v2 ...' text fixture; ints accept 0b prefixes."""
    out = {}
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        parsed = []
        for v in vals:
            try:
                parsed.append(int(v, 0))
            except ValueError:
                parsed.append(float(v))
        out[key] = parsed
    return out


@pytest.fixture(scope="session")
def golden_dialect4():
    return read_golden("dialect4_example.txt")
