import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


def read_golden(name="paper_values.txt"):
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if "=" in line:
                k, v = line.split("=", 1)
                out[k.strip()] = float(v)
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden()


@pytest.fixture(autouse=True)
def parity_stats(request, capsys):
    """GPU tests: one JSON line per test with the worst errors its parity helpers saw."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    import json

    import parity_utils as PU
    PU.STATS.clear()
    yield
    if PU.STATS:
        with capsys.disabled():
            print("\nPARITY " + json.dumps({"test": request.node.nodeid, "worst": PU.STATS}, sort_keys=True))
