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
    """Near-threshold counts and worst errors of every GPU/oracle comparison of the run."""
    try:
        import parity
    except Exception:
        return
    if not parity.REPORT:
        return
    terminalreporter.write_line("parity against the CPU oracle (near = decisions that differ with the "
                                "deciding score inside its tolerance; worst = largest errors seen):")
    for r in parity.REPORT:
        terminalreporter.write_line(f"  {r['label']}: seqs={r['seqs']} near={r['near']} worst={r['worst']}")
