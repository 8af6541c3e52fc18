import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


def pytest_terminal_summary(terminalreporter):
    """Near-tie controller decisions (top-two logit gap < 1e-5) are listed separately from the assertions."""
    gu = sys.modules.get("gpu_util")
    if gu is None or not gu.NEAR_TIE_REPORTS:
        return
    terminalreporter.section("controller decisions: near ties")
    for line in gu.near_tie_summary_lines():
        terminalreporter.write_line(line)
