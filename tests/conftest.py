import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    config.addinivalue_line("markers", "slow: full-size case, minutes on the host side")


@pytest.fixture(autouse=True)
def _workspace_guards():
    """After every GPU test: the guard blocks around the last workspace of every cached context must be intact."""
    yield
    gu = sys.modules.get("tests.gpu_util")
    if gu is not None:
        gu.check_all_guards()
