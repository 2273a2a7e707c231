import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def c1():
    import synth_inputs as si
    return si.CONFIGS["c1"]


@pytest.fixture(scope="session")
def c1_weights(c1):
    import synth_inputs as si
    return si.all_weights(c1)
