import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
if os.path.dirname(os.path.abspath(__file__)) not in sys.path:
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200, sm_100a)")


def pytest_terminal_summary(terminalreporter):
    """Excuse counts of every lockstep parity run, so that they show in the test output."""
    try:
        import parity_util
    except Exception:
        return
    if parity_util.REPORT:
        terminalreporter.write_sep("-", "parity: logit error, excused and mismatching decisions per run")
        for line in parity_util.REPORT:
            terminalreporter.write_line(line)
