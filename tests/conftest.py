import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


def pytest_sessionfinish(session, exitstatus):
    """With QD_PARITY_LOG=<file>: dump the error figures the GPU parity tests collected (max-normalised, rms-relative,
    worst sequence) as JSON."""
    path = os.environ.get("QD_PARITY_LOG")
    if not path:
        return
    try:
        import json
        import gpu_util
    except Exception:
        return
    if gpu_util.LOG:
        with open(path, "w") as f:
            json.dump([dict(zip(("label", "tensor", "max", "rms", "per_seq"), r)) for r in gpu_util.LOG], f, indent=0)
