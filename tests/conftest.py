import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def read_golden(name):
    """Parse a `key = v v v` text fixture; numbers become float (or int for 0x.. / integer text)."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = [t.strip() for t in line.split("=", 1)]
            toks = []
            for t in val.split():
                if t.lower().startswith("0x"):
                    toks.append(int(t, 16))
                else:
                    try:
                        toks.append(int(t))
                    except ValueError:
                        toks.append(float(t))
            out[key] = toks
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden
