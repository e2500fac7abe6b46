import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def oracle64():
    from oracle import Oracle
    return Oracle("f64")


@pytest.fixture(scope="session")
def oracle32():
    from oracle import Oracle
    return Oracle("f32")


def pytest_terminal_summary(terminalreporter):
    """Reports the largest value of each parity error measure that the session's GPU comparisons saw."""
    try:
        import helpers
    except Exception:  # noqa: BLE001
        return
    for dtype, (e1, e2, e3) in sorted(helpers.WORST.items()):
        terminalreporter.write_line(
            f"parity error measures, {dtype}: tensor-max-normalised {e1:.3e}, elementwise {e2:.3e}, "
            f"per (row, head) {e3:.3e}")
