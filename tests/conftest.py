import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def load_golden(name):
    """Parse a text fixture under tests/golden/: lines of
    ``NAME rows cols v0 v1 ...`` (row-major), '#' starts a comment."""
    import numpy as np

    out = {}
    path = os.path.join(ROOT, "tests", "golden", name)
    with open(path) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            parts = line.split()
            key, r, c = parts[0], int(parts[1]), int(parts[2])
            vals = np.array([float(v) for v in parts[3:]], dtype=np.float64)
            assert vals.size == r * c, (name, key)
            out[key] = vals.reshape(r, c)
    return out


@pytest.fixture(scope="session")
def golden():
    return load_golden
