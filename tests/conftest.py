import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def load_golden(name):
    """Parse a tests/golden text fixture: 'name rows cols' headers followed by rows of numbers."""
    import numpy as np
    out = {}
    path = os.path.join(ROOT, "tests", "golden", name)
    with open(path) as f:
        lines = [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]
    i = 0
    while i < len(lines):
        key, r, c = lines[i].split()
        r, c = int(r), int(c)
        vals = [[float(v) for v in lines[i + 1 + j].split()] for j in range(r)]
        out[key] = np.array(vals, dtype=np.float64).reshape(r, c)
        i += 1 + r
    return out
