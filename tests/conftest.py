import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a) and the built library")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """How often a parity comparison had to accept the kernel's slot order for (nearly) tied
    coefficients instead of the oracle's (see parity_util.py)."""
    try:
        import parity_util
    except Exception:  # pragma: no cover
        return
    if not parity_util.SLOT_TALLY:
        return
    tr = terminalreporter
    tr.write_sep("-", "slot order of Eq. 11: workers that took a swapped slot (near-ties)")
    tot = [0, 0, 0]
    for what, (steps, sets, swapped) in sorted(parity_util.SLOT_TALLY.items()):
        tot = [tot[0] + steps, tot[1] + sets, tot[2] + swapped]
        if swapped:
            tr.write_line(f"  {what}: {swapped} workers over {steps} steps / {sets} coefficient sets")
    tr.write_line(f"  total: {tot[2]} workers over {tot[0]} steps / {tot[1]} coefficient sets compared; "
                  f"{sum(1 for v in parity_util.SLOT_TALLY.values() if v[2] == 0)} of {len(parity_util.SLOT_TALLY)} "
                  "cases needed no swap")
