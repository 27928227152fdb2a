import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


def pytest_sessionstart(session):
    """Bring the in-tree library up to date with its sources before anything loads it (a no-op when it is; the binding
    itself never builds and refuses to run without the library)."""
    try:
        from paper_2609_14507_b200 import build
        if os.path.exists(build.NVCC):
            build.build()
            build.build(checked=True)
    except Exception as e:                                  # the tests that need the library will say so themselves
        sys.stderr.write(f"conftest: could not build libipkv.so: {e}\n")


def read_golden(name="paper_tables.txt"):
    """key -> float from a ``tests/golden`` text fixture."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, val = line.split("=")
            out[key.strip()] = float(val)
    return out


@pytest.fixture(scope="session")
def golden():
    return read_golden()
