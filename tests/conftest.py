import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def load_golden(name):
    """Parse a `name = hex` fixture; a value may continue on following indented lines."""
    out, key = {}, None
    with open(os.path.join(GOLDEN, name)) as f:
        for raw in f:
            line = raw.rstrip("\n")
            if not line.strip() or line.lstrip().startswith("#"):
                continue
            if "=" in line and not line[0].isspace():
                key, val = line.split("=", 1)
                key = key.strip()
                out[key] = val.strip()
            else:
                out[key] += line.strip()
    return {k: bytes.fromhex(v) for k, v in out.items()}


@pytest.fixture(scope="session")
def golden():
    return load_golden
