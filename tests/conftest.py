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
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


def pytest_terminal_summary(terminalreporter):
    """The parity figures of the GPU tests: per compared step the worst relative L2 error against the plain oracle and
    against the oracle evaluated under the GPU's in-window ReLU decisions (a diagnostic), with the decision counts."""
    try:
        import hpf_testlib
    except Exception:
        return
    if hpf_testlib.PARITY_LOG:
        terminalreporter.write_sep("-", "parity against the fp64 oracle")
        for line in hpf_testlib.PARITY_LOG:
            terminalreporter.write_line(line)
