import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle

    _oracle.build()
    return _oracle


def pytest_terminal_summary(terminalreporter):
    """The parity reports of the GPU tests (score error, order differences with their oracle gaps,
    tie margins, allocation differences), printed whether or not output is captured."""
    try:
        import parity
    except Exception:  # noqa: BLE001
        return
    if not parity.REPORTS:
        return
    terminalreporter.section("parity reports (GPU vs the all-double oracle)")
    for name, fields in parity.REPORTS:
        terminalreporter.write_line("%s: %s" % (name, ", ".join("%s=%s" % kv for kv in fields.items())))
