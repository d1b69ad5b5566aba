import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def read_golden(name):
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = (s.strip() for s in line.split("=", 1))
            out[k] = float(v)
    return out


@pytest.fixture(scope="session")
def worked_example():
    return read_golden("worked_example.txt")


@pytest.fixture(scope="session")
def pdlib():
    """The Python binding, after (re)building libpd.so in-tree if it is missing or stale."""
    import subprocess
    res = subprocess.run([sys.executable, os.path.join(ROOT, "paper_2603_04716_b200", "build.py")],
                         capture_output=True, text=True)
    assert res.returncode == 0, res.stdout + res.stderr
    import paper_2603_04716_b200 as pd
    return pd
