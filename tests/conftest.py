import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


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


# ---------------------------------------------------------------- parity report
# Tests that compare the CUDA path with the oracle record the figures they measured (literal errors,
# fractions of differing codes, how much each allowance was used) with record_parity(); the session
# prints them and, if FP8MLP_PARITY_REPORT names a file, writes them there as JSON.
from helpers import PARITY_FIGURES as _PARITY  # noqa: E402


def pytest_terminal_summary(terminalreporter):
    if not _PARITY:
        return
    import json
    terminalreporter.write_sep("-", "parity figures")
    for row in _PARITY:
        terminalreporter.write_line(json.dumps(row))
    path = os.environ.get("FP8MLP_PARITY_REPORT")
    if path:
        with open(path, "w") as fh:
            json.dump(_PARITY, fh, indent=1)
