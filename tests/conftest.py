import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a); run with -m gpu on a B200")


def load_golden(name):
    """Parse a tests/golden text fixture: blocks of 'name rows cols' followed by the rows."""
    import numpy as np
    out = {}
    path = os.path.join(ROOT, "tests", "golden", name)
    with open(path) as fh:
        lines = [ln.strip() for ln in fh if ln.strip() and not ln.lstrip().startswith("#")]
    i = 0
    while i < len(lines):
        key, rows, cols = lines[i].split()
        rows, cols = int(rows), int(cols)
        vals = [[float(v) for v in lines[i + 1 + r].split()] for r in range(rows)]
        arr = np.asarray(vals, dtype=np.float64).reshape(rows, cols)
        out[key] = arr
        i += 1 + rows
    return out


@pytest.fixture(scope="session")
def golden_example():
    return load_golden("worked_example.txt")
