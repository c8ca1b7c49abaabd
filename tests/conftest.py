import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


# Lines that tests want in the run's output even when they pass and output is captured (the
# sample a full-size parity test compared, its counts): printed in the terminal summary.
_REPORT_LINES = []


def report_line(text: str) -> None:
    _REPORT_LINES.append(text)
    print(text)


def pytest_terminal_summary(terminalreporter):
    if _REPORT_LINES:
        terminalreporter.section("parity samples")
        for line in _REPORT_LINES:
            terminalreporter.write_line(line)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); runs the CUDA library")


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
