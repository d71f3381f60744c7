import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def load_golden(name):
    """Parse a 'key v v v' text fixture from tests/golden into {key: [floats]}."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(t) for t in v]
    return out


@pytest.fixture(scope="session")
def hand4():
    return load_golden("hand_4x4.txt")


@pytest.fixture(scope="session")
def hand_blocks4():
    return load_golden("hand_blocks_4x4.txt")
