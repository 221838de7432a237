import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu)")


@pytest.fixture(scope="session")
def orc():
    import oracle
    oracle.build()
    return oracle


def pytest_terminal_summary(terminalreporter):
    """Shares of margin-rule decisions recorded by the parity tests (shown whether or not output is captured)."""
    try:
        import parity_util
    except ImportError:
        return
    if parity_util.REPORT:
        terminalreporter.write_sep("-", "decisions inside the oracle's margins")
        for line in parity_util.REPORT:
            terminalreporter.write_line(line)
