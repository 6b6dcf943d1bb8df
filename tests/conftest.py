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
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """How many compared elements were above 1e-2, for decode and for prefill."""
    try:
        import helpers
    except Exception:  # pragma: no cover
        return
    t = helpers.TALLY
    if not t["calls"]:
        return
    terminalreporter.write_line(
        f"parity tally: {t['calls']} comparisons with the oracle, {t['elements']} elements "
        f"({t['amended_elements']} of them prefill outputs under the amended bound); "
        f"decode: {t['decode_over_abs_tol']} of {t['decode_elements']} elements above 1e-2"
        + (f" (all of magnitude >= {t['decode_over_min_ref']:.3f}, where half a bf16 spacing "
           f"is 1.56e-2)" if t["decode_over_abs_tol"] else "")
        + f"; prefill: {t['over_abs_tol']} elements above 1e-2"
        + (f" (smallest |ref| {t['over_abs_tol_min_ref']:.3f}, largest error "
           f"{t['over_abs_tol_max_err']:.4e}): " + "; ".join(t["over_abs_tol_where"])
           if t["over_abs_tol"] else ""))
