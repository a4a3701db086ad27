import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_sessionstart(session):
    """Build the C-ABI library when it is missing (nvcc cross-compiles without a GPU).  The package
    itself never builds or falls back: it raises when the library is absent."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("_fedattn_build", os.path.join(ROOT, "paper_2511_02647_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    if not os.path.exists(mod.LIB_PATH):
        mod.build()


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle
