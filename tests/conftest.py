import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def load_golden():
    """Values the paper prints (tests/golden/paper_values.txt: name | value | where it is printed)."""
    vals = {}
    with open(os.path.join(ROOT, "tests", "golden", "paper_values.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, value, _where = [x.strip() for x in line.split("|", 2)]
            vals[name] = int(value)
    return vals


@pytest.fixture(scope="session")
def golden():
    return load_golden()
