import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (the parity tests proper)")


@pytest.fixture(scope="session")
def golden():
    """Values printed in the paper: name -> (float value, citation)."""
    out = {}
    path = os.path.join(ROOT, "tests", "golden", "paper_constants.txt")
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, value, cite = line.split("|")
            out[name.strip()] = (float(value), cite.strip())
    return out
