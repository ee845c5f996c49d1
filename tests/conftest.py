import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """Every GPU test gets a wall-clock limit (when pytest-timeout is installed): a kernel that
    never returns must end the test, not the session."""
    if not config.pluginmanager.hasplugin("timeout"):
        return
    for item in items:
        if item.get_closest_marker("gpu") and not item.get_closest_marker("timeout"):
            item.add_marker(pytest.mark.timeout(300))


def read_golden(name):
    """Parse a tests/golden fixture: '#' lines are comments (the citation),
    'key: v v v' lines give integer or float lists."""
    out = {}
    path = os.path.join(ROOT, "tests", "golden", name)
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":")
            out[key.strip()] = [float(v) if "." in v else int(v) for v in vals.split()]
    return out


@pytest.fixture
def golden():
    return read_golden
