import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


@pytest.fixture(scope="session")
def golden_dir():
    return GOLDEN


@pytest.fixture
def test_build(monkeypatch):
    """Every library call inside the test goes to the test build (libspecblock_test.so): the same
    sources plus the mma.sync / one-warp-per-row check kernels and the environment switches that
    force a kernel variant.  Yields monkeypatch, for setting those switches."""
    from paper_2605_07243_b200 import binding as sb
    with sb.build_variant("test"):
        yield monkeypatch
