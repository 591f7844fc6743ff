import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def load_rational_fixture(name):
    """Parse tests/golden/<name>: 'label rows cols' headers followed by rationals."""
    from fractions import Fraction
    import numpy as np
    path = os.path.join(ROOT, "tests", "golden", name)
    toks = []
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0]
            toks.extend(line.split())
    out, i = {}, 0
    while i < len(toks):
        label, r, c = toks[i], int(toks[i + 1]), int(toks[i + 2])
        vals = [Fraction(t) for t in toks[i + 3:i + 3 + r * c]]
        out[label] = np.array([float(v) for v in vals]).reshape(r, c)
        i += 3 + r * c
    return out


@pytest.fixture(scope="session")
def worked_example():
    return load_rational_fixture("worked_example.txt")
