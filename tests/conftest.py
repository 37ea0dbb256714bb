import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def tiny_shape():
    import ppd_inputs
    return ppd_inputs.TINY


@pytest.fixture(scope="session")
def tiny_blob(tiny_shape):
    import ppd_inputs
    return ppd_inputs.gen_weights(tiny_shape, seed=0)


@pytest.fixture(scope="session")
def tiny_prompt(tiny_shape):
    import ppd_inputs
    return ppd_inputs.gen_prompt(tiny_shape.vocab, 16, seed=1)


def read_golden(name):
    """Parse tests/golden/<name>: 'key = value  # citation' lines."""
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            k, v = line.split("=", 1)
            out[k.strip()] = v.strip()
    return out
