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
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


# Lines the parity tests want shown even under `-q` (sample sizes, excused counts, worst errors): they are
# printed in the terminal summary and, when CRISP_PARITY_SUMMARY names a file, appended to it.
_PARITY_LINES = []


@pytest.fixture
def parity_report():
    return _PARITY_LINES.append


def pytest_terminal_summary(terminalreporter):
    if not _PARITY_LINES:
        return
    terminalreporter.section("parity summary")
    for line in _PARITY_LINES:
        terminalreporter.write_line(line)
    path = os.environ.get("CRISP_PARITY_SUMMARY")
    if not path:
        return
    try:
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        with open(path, "a") as f:
            f.write("\n".join(_PARITY_LINES) + "\n")
    except OSError:  # pragma: no cover
        pass
