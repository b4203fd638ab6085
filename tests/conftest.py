import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


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
