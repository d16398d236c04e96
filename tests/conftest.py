import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (runs the CUDA library)")


def read_golden(name):
    """Parse a tests/golden/*.txt fixture: '#' comments, 'key: ints' lines and
    bare rows of integers (returned under key 'rows')."""
    path = os.path.join(ROOT, "tests", "golden", name)
    out = {"rows": []}
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if ":" in line:
                key, val = line.split(":", 1)
                nums = [int(v) for v in val.split()]
                out[key.strip()] = nums[0] if len(nums) == 1 else nums
            else:
                out["rows"].append([int(v) for v in line.split()])
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
