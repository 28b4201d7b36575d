import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_collection_modifyitems(config, items):
    """Without a CUDA device the GPU tests are skipped -- unless the run asked for them (`-m gpu`):
    then they stay in and fail, so that a GPU run on a box whose CUDA context did not come up cannot
    pass with every parity test skipped."""
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    asked = (config.getoption("-m") or "").replace(" ", "")
    if "gpu" in asked and "notgpu" not in asked:
        def no_device():
            pytest.fail("this run selected the GPU tests (-m gpu) but no CUDA device is available")
        for item in items:
            if "gpu" in item.keywords:
                item.obj = no_device            # fail, do not skip
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
