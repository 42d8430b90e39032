import json
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


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


_PARITY = {}


@pytest.fixture
def parity_record():
    """record(name, value): keeps a measured parity error.  When the environment variable BETTY_PARITY_LOG names
    a file, the session merges all recorded errors into it as JSON (the figures quoted in the documentation
    come from such a file)."""
    def record(name, value):
        _PARITY[name] = float(value)
        return float(value)
    return record


def pytest_sessionfinish(session, exitstatus):
    path = os.environ.get("BETTY_PARITY_LOG")
    if not _PARITY or not path:
        return
    try:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        old = {}
        if os.path.exists(path):
            with open(path) as f:
                old = json.load(f)
        old.update(_PARITY)
        with open(path, "w") as f:
            json.dump(old, f, indent=1, sort_keys=True)
    except OSError:
        pass
