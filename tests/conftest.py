import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session", autouse=True)
def _built_oracle():
    """The C oracle is compiled on demand (gcc); building the checker is not using it."""
    from oracle import build
    build.build()


@pytest.fixture(scope="session", autouse=True)
def _parity_record():
    """GPU parity tests append the maxima they achieved (not only pass/fail) to a JSON-lines record: the file
    named by PODS_PARITY_RECORD, else parity_maxima.jsonl in pytest's cache folder."""
    import parity
    path = os.environ.get("PODS_PARITY_RECORD") or os.path.join(ROOT, ".pytest_cache", "parity_maxima.jsonl")
    try:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        parity.RECORD_PATH = path
    except OSError:
        parity.RECORD_PATH = None
    yield
