import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a kernels through the C ABI)")
    config.addinivalue_line("markers", "expired_waits: the test makes bounded waits run out on purpose")


@pytest.fixture(autouse=True)
def _no_bounded_wait_ran_out(request):
    """Every GPU test doubles as a check that none of the staged kernels' bounded waits expired
    (the library counts them per process; the one test that provokes them is marked)."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    from paper_2010_04902_b200 import binding as bz
    before = bz.pipeline_timeouts()
    yield
    if request.node.get_closest_marker("expired_waits") is None:
        assert bz.pipeline_timeouts() == before, "a bounded barrier wait ran out during this test"


@pytest.fixture(scope="session")
def golden_dir():
    return GOLDEN


def read_golden_rows(name):
    """Non-comment lines of a golden text fixture, split on whitespace."""
    rows = []
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows
