import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


# Small calls skip the quick kernel by default; the GPU tests are small, so they lower the limit to
# zero to keep exercising both kernels (tests of the default behaviour unset it again).
os.environ.setdefault("DAF_QUICK_MIN_WINDOWS", "0")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture
def default_quick_limit(monkeypatch):
    """The library's own limit on the windows of a call that goes to the full kernel alone."""
    monkeypatch.delenv("DAF_QUICK_MIN_WINDOWS", raising=False)


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
