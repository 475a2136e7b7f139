import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def read_golden(name):
    """Parse tests/golden/<name>: '#' comments, 'case <id>' headers, 'key: v v v' lines."""
    cases, cur = {}, None
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            if line.startswith("case "):
                cur = {}
                cases[line[5:].strip()] = cur
                continue
            key, _, rest = line.partition(":")
            cur[key.strip()] = [int(t) for t in rest.split()]
    return cases


@pytest.fixture(scope="session")
def golden():
    return read_golden
