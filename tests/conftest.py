import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


@pytest.fixture(autouse=True)
def _reset_debug_knobs():
    """Forced launch geometries (qmm_debug_config) never leak from one test into the next."""
    yield
    mod = sys.modules.get("paper_2607_00501_b200.qmm")
    if mod is not None and mod._lib is not None:
        mod.debug_config(None)
