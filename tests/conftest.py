import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def f64(t):
    """Exact up-cast of a torch tensor (any float dtype, any device) to a float64 numpy array."""
    if t is None:
        return None
    return t.detach().to("cpu").double().numpy()


@pytest.fixture(scope="session")
def rng():
    return np.random.default_rng(20240104)
