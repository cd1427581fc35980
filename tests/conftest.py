import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


# Small calls go to the general compress kernel alone by default; the GPU tests are small, so their
# parameter blocks ask for the streaming kernel whatever the size (tests of the default policy undo it).
import paper_2507_07149_b200 as _daf  # noqa: E402

_daf.DEFAULT_FLAGS = _daf.FLAG_STREAM_ALWAYS


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture
def default_quick_limit(monkeypatch):
    """The library's own rule for which calls go to the general kernel alone."""
    monkeypatch.setattr(_daf, "DEFAULT_FLAGS", 0)


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
