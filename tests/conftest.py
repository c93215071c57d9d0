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
    """What the parity tolerances let through in this run (never silently): see tests/util.py."""
    try:
        import util
    except Exception:
        return
    c = util.COUNTS
    if c["halt_checked"]:
        terminalreporter.write_line(
            f"parity exemptions: halt flags {c['halt_exempt']} of {c['halt_checked']} within {util.HALT_MARGIN:g} of tau "
            f"({c['halt_exempt_differs']} of them differ from the oracle); arg-max near-ties {c['argmax_near_tie']} draft, "
            f"{c['verify_rows_near_tie']} verification rows; max |C_gpu - C_oracle| = {c['max_conf_err']:.2e}")
