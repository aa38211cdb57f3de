import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session", params=["fp16", "int8"])
def codebooks(request):
    """Lloyd-Max codebooks per head_dim from the oracle-side tool, in the two forms the decode kernel accepts: levels
    that are exact binary16 values (fp16 tensor-core path) and levels on an 8-bit grid (integer tensor-core path).
    Every test that takes this fixture runs once per form."""
    from oracle import lloyd_max

    make = lloyd_max.fp16_codebook if request.param == "fp16" else lloyd_max.int8_codebook
    cbs = {d: make(d) for d in (128, 256)}
    cbs["kind"] = request.param
    return cbs
