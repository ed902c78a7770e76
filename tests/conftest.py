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


def read_golden(name):
    """Parse tests/golden/<name>: blocks of '<key> <dims...>' followed by rows of numbers."""
    import numpy as np
    path = os.path.join(ROOT, "tests", "golden", name)
    out, key, dims, buf = {}, None, None, []
    def flush():
        if key is not None:
            out[key] = np.array(buf, dtype=np.float64).reshape(dims)
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0][0].isalpha():
            flush()
            key, dims, buf = tok[0], [int(t) for t in tok[1:]], []
        else:
            buf.extend(float(t) for t in tok)
    flush()
    return out
