import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle():
    """The CPU oracle front end (builds the C library on first use)."""
    from oracle import ref
    ref.lib()
    return ref


@pytest.fixture(scope="session")
def b2():
    """The ctypes binding of the CUDA library (built on demand; no fallback)."""
    from paper_1611_08035_b200 import binding, build
    if not binding.LIB_PATH.exists():
        build.build()
    binding.lib()
    return binding
