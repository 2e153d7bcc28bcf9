import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def pytest_terminal_summary(terminalreporter):
    """Realised float errors of the GPU parity checks: written to parity_errors.json in the output folder and summarised."""
    sys.path.insert(0, str(Path(__file__).resolve().parent))
    import parity_util
    table = parity_util.dump()
    if table:
        terminalreporter.write_sep("-", "realised parity errors (worst case per tensor)")
        terminalreporter.write_line(table)
