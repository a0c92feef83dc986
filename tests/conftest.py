import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


def pytest_terminal_summary(terminalreporter):
    from tests import helpers

    if helpers.OBSERVED_ROW_ERRORS:
        terminalreporter.write_line(
            "worst element error per row (units of the row's RMS), largest over %d checks: %.4f (bound %.2f)"
            % (len(helpers.OBSERVED_ROW_ERRORS), max(helpers.OBSERVED_ROW_ERRORS), helpers.TOL_ROW))
