import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, when no device is present and -m gpu was not asked for."""
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


def read_golden_matrices(path):
    import numpy as np

    out, name, rows, shape = {}, None, [], None
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            if line.startswith("@"):
                if name:
                    out[name] = np.array(rows, dtype=np.float64).reshape(shape)
                parts = line[1:].split()
                name, shape, rows = parts[0], (int(parts[1]), int(parts[2])), []
            else:
                rows.append([float(v) for v in line.split()])
    if name:
        out[name] = np.array(rows, dtype=np.float64).reshape(shape)
    return out


GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
