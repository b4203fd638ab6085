import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session", autouse=True)
def _built_library():
    """Build the CUDA library and the C checker in-tree when they are missing or older than
    their sources (nvcc cross-compiles without a GPU); a failed build fails the session loudly."""
    from paper_2412_01195_b200 import build as dt8_build
    dt8_build.build_library()
    import oracle
    oracle.build()
    yield


def load_paper_facts():
    facts = {}
    path = os.path.join(ROOT, "tests", "golden", "paper_facts.txt")
    with open(path) as fh:
        for line in fh:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, val = (s.strip() for s in line.split("=", 1))
            facts[key] = float(val)
    return facts


@pytest.fixture(scope="session")
def paper_facts():
    return load_paper_facts()
