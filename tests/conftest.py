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
    """GPU parity tests append the maxima they achieved (not only pass/fail) to gpurun_out/parity_maxima.jsonl."""
    import parity
    out = os.path.join(ROOT, "gpurun_out")
    try:
        os.makedirs(out, exist_ok=True)
        parity.RECORD_PATH = os.path.join(out, "parity_maxima.jsonl")
    except OSError:
        parity.RECORD_PATH = None
    yield
