import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: test needs a CUDA device (sm_100a) and the built CUDA library")


def pytest_sessionstart(session):
    """Build the CUDA library when it is missing or older than its sources (a no-op otherwise), so that a fresh
    checkout can run the suite directly.  A failed build is not hidden: the tests that need the library fail."""
    try:
        from paper_2603_19664_b200.build import build
        build()
        build(check=True)  # the checking build (device-side index tests), used by tests/test_gpu_check_build.py
    except Exception as e:  # noqa: BLE001
        sys.stderr.write(f"[conftest] building libkvd.so failed: {e}\n")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")
