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


def pytest_terminal_summary(terminalreporter, exitstatus, config):
    """The plain bf16 bar (max|err| <= 2e-2 * RMS(ref)) per compared tensor, next to the asserted tolerances:
    the worst ratio seen and how many elements exceed the plain bar."""
    try:
        from tests.util import PARITY_LOG
    except Exception:
        return
    if not PARITY_LOG:
        return
    worst = {}
    for what, ratio, n_over, n in PARITY_LOG:
        key = what.split("[")[0].strip()
        r0, o0, n0 = worst.get(key, (0.0, 0, 0))
        worst[key] = (max(r0, ratio), o0 + n_over, n0 + n)
    tr = terminalreporter
    tr.write_sep("-", "plain bf16 metric: max|err| / RMS(ref) per tensor (bar 2e-2), elements over it")
    for key in sorted(worst):
        r, o, n = worst[key]
        tr.write_line(f"{key:32s} {r:8.4f}   over: {o} of {n}")
