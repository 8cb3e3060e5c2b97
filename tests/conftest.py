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
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(scope="session")
def flashd_lib():
    """Build (if stale) and load the C-ABI CUDA library."""
    from paper_2505_14201_b200 import build as _build
    _build.build()
    import paper_2505_14201_b200 as pkg
    pkg.lib()
    return pkg


def read_golden(name):
    """Parse a ``key: v v v`` text fixture into {key: [Fraction, ...]}."""
    from fractions import Fraction
    out = {}
    with open(os.path.join(ROOT, "tests", "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, vals = line.split(":", 1)
            out[key.strip()] = [Fraction(t) for t in vals.split()]
    return out
