import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def codebooks():
    """fp16-representable Lloyd-Max codebooks per head_dim, from the oracle-side tool."""
    from oracle import lloyd_max

    return {d: lloyd_max.fp16_codebook(d) for d in (128, 256)}
