import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session", autouse=True)
def _oracle_threads():
    # The oracle's loops over independent outputs may use every host core; results do
    # not depend on the thread count.
    from oracle import binding
    binding.set_threads(os.cpu_count() or 1)
    yield


@pytest.fixture(autouse=True)
def _parity_context(request):
    # value comparisons made during a test are recorded under the test's name
    from tests import harness
    harness.parity_context(request.node.name)
    yield
    harness.parity_context("")


def pytest_terminal_summary(terminalreporter):
    """Measured errors of every value comparison of the run (max|err|/rms, rms(err)/rms, elements
    beyond 2e-2*rms): printed, and written as tab-separated text to $ETR_PARITY_REPORT if set."""
    try:
        from tests import harness
    except Exception:
        return
    log = harness.PARITY_LOG
    if not log:
        return
    lines = ["comparison\telements\tmax_err_over_rms\trms_err_over_rms\tbeyond_2e-2_rms"]
    lines += [f"{w}\t{n}\t{mx:.3e}\t{rm:.3e}\t{nb}" for w, n, mx, rm, nb in log]
    path = os.environ.get("ETR_PARITY_REPORT")
    if path:
        with open(path, "w") as f:
            f.write("\n".join(lines) + "\n")
    worst = sorted(log, key=lambda r: -r[2])[:12]
    terminalreporter.write_line("largest max|err|/rms(ref) among the value comparisons of this run:")
    for w, n, mx, rm, nb in worst:
        terminalreporter.write_line(f"  {w}: max {mx:.3e}  rms {rm:.3e}  beyond 2e-2: {nb} of {n}")
