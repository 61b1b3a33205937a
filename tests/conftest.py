import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (sm_100a)")


@pytest.fixture(scope="session")
def dsn():
    """The ctypes binding of the CUDA library; GPU tests fail loudly when it is missing."""
    import paper_2109_10060_b200 as pkg
    return pkg


# Measured parity figures (worst errors per configuration) that the GPU tests want shown with the result.
PARITY_REPORT = []


@pytest.fixture(scope="session")
def parity_report():
    return PARITY_REPORT


def pytest_terminal_summary(terminalreporter):
    if PARITY_REPORT:
        terminalreporter.write_line("measured parity figures (max|err| / max|ref| per group unless stated):")
        for line in PARITY_REPORT:
            terminalreporter.write_line("  " + line)
