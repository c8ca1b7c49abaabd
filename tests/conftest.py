import os
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
    if _GUARDED is not None:
        terminalreporter.section("bounds-checked library")
        terminalreporter.write_line(
            f"[debug sweep] {_SWEEP['tests']} tests under the bounds-checked library: "
            f"{_SWEEP['violations']} index violations, {_GUARDED.regions_checked} guard regions intact")


# ---- the debug sweep: A2SF_LIBRARY=debug selects the bounds-checked library (binding.py) and
# A2SF_GUARDS=1 puts canary words around everything the binding and the harness allocate; after
# every test the library must report zero index violations and every guard must be intact.
_GUARDED = None
_SWEEP = {"tests": 0, "violations": 0}


@pytest.fixture(autouse=True)
def _debug_sweep(request):
    global _GUARDED
    if os.environ.get("A2SF_GUARDS", "") != "1" or "gpu" not in request.keywords:
        yield
        return
    import torch

    import parity_util
    from guards import GuardedTorch
    from paper_2407_20485_b200 import binding

    if _GUARDED is None:
        assert binding.a2sf_debug_build(), "A2SF_GUARDS=1 expects A2SF_LIBRARY=debug"
        _GUARDED = GuardedTorch(torch)
        binding.torch = _GUARDED              # every allocation of the binding ...
        parity_util.torch = _GUARDED          # ... and of the parity harness gets guard words
        for name in ("test_parity_gpu", "test_policies"):        # ... and of the test modules themselves
            if name in sys.modules:
                sys.modules[name].torch = _GUARDED
    binding.a2sf_debug_violations()           # start from a clean record
    yield
    torch.cuda.synchronize()
    count, kernel, line, index, bound = binding.a2sf_debug_violations()
    _SWEEP["tests"] += 1
    _SWEEP["violations"] += count
    assert count == 0, (f"{count} out-of-range indices inside kernels; first: kernel id {kernel}, source line "
                        f"{line}, index {index}, bound {bound}")
    _GUARDED.check(request.node.name)
    _GUARDED.release()


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
