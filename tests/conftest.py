import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


@pytest.fixture(scope="session", autouse=True)
def _build_cpu_libs():
    """The generator and the C part of the oracle are plain gcc builds; make sure they exist."""
    import gen
    import oracle
    gen.build()
    oracle.build()


def pytest_terminal_summary(terminalreporter):
    """Worst error any parity comparison of this session saw, under the asserted metric and the two recorded ones."""
    try:
        import parity_util
    except ImportError:
        return
    if any(parity_util.SESSION_WORST.values()):
        terminalreporter.write_line("parity, worst error of the session by metric: " +
                                    ", ".join(f"{k} {v:.3g}" for k, v in parity_util.SESSION_WORST.items()))
