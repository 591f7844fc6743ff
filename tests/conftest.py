import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_sessionfinish(session, exitstatus):
    """After a GPU session: the three error figures of every comparison with the oracle, worst case per tensor
    name and dtype, as a text table in the run's output folder (written only where that folder exists)."""
    try:
        from parity import parity_report
    except ImportError:
        return
    out_dir = os.path.join(ROOT, "gpurun_out")
    if not parity_report or not os.path.isdir(out_dir):
        return
    worst = {}
    for what, dtype, shape, row, gated, rms in parity_report:
        import re
        key = (re.sub(r"(, length|step) \d+", r"\1 *", what.split("[")[0]), dtype)
        w = worst.setdefault(key, [0.0, 0.0, 0.0, 0])
        w[0], w[1], w[2], w[3] = max(w[0], row), max(w[1], gated), max(w[2], rms), w[3] + 1
    with open(os.path.join(out_dir, "parity_report.txt"), "w") as f:
        f.write("tensor dtype comparisons row gated rms   (maxima over all comparisons of the session)\n")
        for (what, dtype), (row, gated, rms, n) in sorted(worst.items()):
            f.write(f"{what or '-'} {dtype} {n} {row:.3e} {gated:.3e} {rms:.3e}\n")


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
