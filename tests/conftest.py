import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


@pytest.fixture(autouse=True)
def _guard_bands(request, monkeypatch):
    """GPU tests: every buffer obtained through the package's empty_global lies between guard bands
    (tests/helpers.py), and the bands are checked when the test ends."""
    if request.node.get_closest_marker("gpu") is None:
        yield
        return
    import helpers
    import paper_2110_15032_b200 as sbp
    monkeypatch.setattr(sbp, "empty_global", helpers.guarded_empty_global)
    helpers._GUARDED.clear()
    yield
    helpers.check_guards(clear=True)
    sbp.sbp_check_device_errors()     # an expired device wait, or (debug-bounds build) a refused address


GOLDEN = os.path.join(ROOT, "tests", "golden")


def read_golden(name):
    """Non-comment lines of a text fixture, split on whitespace."""
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows
