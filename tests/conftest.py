import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")
    config.addinivalue_line("markers", "slow: minutes of CPU oracle time (deselect with -m 'gpu and not slow')")


def pytest_collection_modifyitems(config, items):
    # tests marked gpu are skipped where no device is visible
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


GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden_values(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            body = line.split("|")[0]
            key, val = body.split("=")
            out[key.strip()] = int(val.strip())
    return out


def read_golden_table2():
    modes = {"R": 0, "S": 1, "S*": 2, "M": 3, "O": 4}
    out = {}
    with open(os.path.join(GOLDEN, "table2_placements.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, spec, role = [p.strip() for p in line.split("|")]
            pis = [modes[t] for t in spec.split()]
            out[name] = (pis[0] + 5 * pis[1] + 25 * pis[2] + 125 * pis[3], role)
    return out
