import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have_gpu = torch.cuda.is_available()
    except Exception:
        have_gpu = False
    if have_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    try:
        from _gpu_util import FP16_ULP_STATS as st
    except Exception:
        return
    if st["compared"]:
        terminalreporter.write_line(
            "fp16 results against the oracle rounded to fp16: %d compared (|ref| >= 0.01 S), "
            "%d beyond one ulp, worst %d ulps" % (st["compared"], st["beyond_one_ulp"], st["worst_ulp"]))
