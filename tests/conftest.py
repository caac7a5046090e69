import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


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


# Counters the parity tests tolerate by protocol (selection swaps between near-equal scores, arg-max
# near-ties, elements on the one-ulp allowance) are part of the result: tests hand their lines to the
# `parity_report` fixture and the lines are printed in the terminal summary, whatever the verbosity.
_PARITY_LINES = []


@pytest.fixture
def parity_report():
    def add(line: str):
        _PARITY_LINES.append(str(line))
        print(line)
    return add


def pytest_terminal_summary(terminalreporter):
    if _PARITY_LINES:
        terminalreporter.section("parity counters (tolerated by protocol, reported)")
        for line in _PARITY_LINES:
            terminalreporter.write_line(line)
