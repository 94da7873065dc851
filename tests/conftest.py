import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def orc():
    """The CPU oracle (compiled with gcc on first use)."""
    from oracle import ampq_oracle

    ampq_oracle.build()
    return ampq_oracle


GOLDEN = os.path.join(ROOT, "tests", "golden")


def read_golden(name):
    """Parse a golden text fixture: 'key = value' lines, '#' comments."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out


@pytest.fixture(scope="session")
def ampq():
    """The ctypes binding of the CUDA library (built with nvcc when stale)."""
    from paper_2505_13060_b200 import binding, build

    if build.needs_build():
        build.build()
    binding.lib()
    return binding
