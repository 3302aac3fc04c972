import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def _tuning_knobs_do_not_leak():
    """A test that pins a launcher choice (binding.set_tuning) must not change what the next test runs."""
    yield
    from paper_1602_06709_b200 import binding as B
    if B._lib is not None:
        B.reset_tuning()


@pytest.fixture(autouse=True)
def _guard_bands_intact():
    """Outputs and workspaces allocated through gpu_helpers sit between pattern-filled bands: no kernel of the test
    may have written outside its buffers."""
    yield
    import sys
    G = sys.modules.get("gpu_helpers")
    if G is not None and G._guards:
        G.check_guards(clear=True)
