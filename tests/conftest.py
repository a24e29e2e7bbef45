import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_collection_modifyitems(config, items):
    # GPU tests are skipped, not failed, on a box without a device.
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


# Observed max |Y_gpu - Y_oracle| / tol per named case, printed after the run: how close each case comes to the bound.
_RATIOS = {}


@pytest.fixture
def ratio_log():
    def log(name, ratio):
        _RATIOS[name] = max(float(ratio), _RATIOS.get(name, 0.0))
        return ratio
    return log


def pytest_terminal_summary(terminalreporter):
    if _RATIOS:
        terminalreporter.write_line("max |dY| / tol per case (bound 1.0):")
        for name in sorted(_RATIOS):
            terminalreporter.write_line(f"  {name}: {_RATIOS[name]:.4g}")
