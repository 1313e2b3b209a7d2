import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


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


def pytest_terminal_summary(terminalreporter):
    # how many compared outputs needed the bound that applies from magnitude 8 on (see test_gpu_parity.py)
    mod = sys.modules.get("test_gpu_parity")
    if mod is not None and getattr(mod, "RELAXED", {}).get("elements"):
        r = mod.RELAXED
        terminalreporter.write_line(
            f"parity: {r['elements']} output element(s) of magnitude >= 8 exceeded the flat 2e-2 bound "
            f"(worst by {r['worst_excess_over_flat']:.3e}); all within bf16 half-ulp + 4.4e-3")
