import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200) and the built library")


def pytest_terminal_summary(terminalreporter):
    """With GRIFFIN_TEST_STATS set, the worst output errors seen by out_check.assert_output over the run (the
    figures its bounds are derived from); GRIFFIN_TEST_STATS=loose also holds the run to the stated bounds only."""
    if os.environ.get("GRIFFIN_TEST_STATS"):
        import json

        import out_check
        terminalreporter.write_line("output error statistics: " + json.dumps(out_check.stats()))
