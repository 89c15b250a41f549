import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def read_golden_blocks(name):
    """Parse a tests/golden text fixture of '# comment', 'label' and number rows."""
    import numpy as np
    blocks, cur = {}, None
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            try:
                row = [float(p) for p in parts]
                blocks[cur].append(row)
            except ValueError:
                cur = parts[0]
                blocks[cur] = []
                if len(parts) > 1:
                    blocks[cur] = [float(p) for p in parts[1:]]
    return {k: np.array(v) for k, v in blocks.items()}
