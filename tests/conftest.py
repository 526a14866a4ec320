import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
HERE = os.path.dirname(os.path.abspath(__file__))
if HERE not in sys.path:
    sys.path.insert(0, HERE)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def tiny_cfg():
    from synthetic import get_config
    return get_config("c0")


@pytest.fixture(scope="session")
def tiny_weights(tiny_cfg):
    from synthetic import draw_weights
    return draw_weights(tiny_cfg)
