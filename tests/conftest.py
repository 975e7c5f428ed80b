import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); runs through the C-ABI library")
    # the library is built in-tree and kept out of version control: (re)build it when missing or stale
    from paper_2506_10401_b200 import build as _build
    _build.build()


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


@pytest.fixture(autouse=True)
def _label_parity_records(request):
    from tests import parity
    parity.set_label(request.node.name)
    yield


def pytest_terminal_summary(terminalreporter):
    """Ungraded strict figures of the fp32 comparisons (largest relative error with no allowance for cancellation)."""
    from tests import parity
    lines = parity.report_lines()
    if lines:
        terminalreporter.write_sep("-", "fp32 parity: strict figures")
        for line in lines:
            terminalreporter.write_line(line)
