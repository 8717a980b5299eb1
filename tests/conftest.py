import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as orc
    orc.build()
    return orc


@pytest.fixture(scope="session")
def lgn():
    """The CUDA library's Python binding (builds the shared library if the
    in-tree copy is missing or older than its sources)."""
    from paper_2006_08173_b200 import build as _build
    _build.build()
    from paper_2006_08173_b200 import binding
    return binding


GOLDEN = os.path.join(ROOT, "tests", "golden")


def golden_lines(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                rows.append(line.split())
    return rows
