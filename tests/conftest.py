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
    """Observed output errors of the GPU parity cases (max|dy|/rms of the returned tensors)."""
    try:
        import parity
    except Exception:
        return
    if not parity.LAST:
        return
    bf = [c for c in parity.LAST if c["dtype"] == "bf16"]
    f32 = [c for c in parity.LAST if c["dtype"] == "f32"]
    if bf:
        worst = max(bf, key=lambda c: c["max_err_over_rms"])
        n_ulp = sum(c["needed_half_ulp"] for c in bf)
        n_el = sum(c["elements"] for c in bf)
        terminalreporter.write_line(
            f"parity: {len(bf)} bf16 output checks, worst max|dy|/rms of a returned bf16 tensor "
            f"{worst['max_err_over_rms']:.3e} {worst['what']}; {n_ulp} of {n_el} elements were beyond "
            f"2e-2 rms and within the half-ulp term")
    if f32:
        worst = max(f32, key=lambda c: c["max_err_over_rms"])
        terminalreporter.write_line(f"parity: {len(f32)} fp32 output checks, worst max|dy|/rms "
                                    f"{worst['max_err_over_rms']:.3e} {worst['what']}")
