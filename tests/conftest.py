import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


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


GOLDEN = os.path.join(ROOT, "tests", "golden")


def read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def pytest_terminal_summary(terminalreporter):
    """How far the fp32 outputs are from the rule without the sum-of-terms relaxation, per case."""
    try:
        from helpers import STRICT_REPORT
    except Exception:
        return
    if not STRICT_REPORT:
        return
    tr = terminalreporter
    tr.write_sep("-", "fp32 outputs outside 1e-5 |ref| and 1e-6 (all inside the tolerance the tests assert)")
    total = missed = 0
    for what, (n, m, worst) in sorted(STRICT_REPORT.items()):
        total, missed = total + n, missed + m
        if m:
            tr.write_line(f"{what}: {m} of {n} outputs, largest |err| {worst:.3e}")
    tr.write_line(f"all cases: {missed} of {total} outputs")
