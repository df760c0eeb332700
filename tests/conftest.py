import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


GOLDEN = os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="session")
def golden_dir():
    return GOLDEN


def pytest_sessionfinish(session, exitstatus):
    """With DYN_CHECKED=1 the tests run against the checking build of the library: at the end of the session the
    index checks of all kernels must have recorded nothing."""
    if os.environ.get("DYN_CHECKED", "") in ("", "0"):
        return
    try:
        import torch
        if not torch.cuda.is_available():
            return
        import paper_2408_00741_b200 as dyn
        status = dyn.dyn_debug_status()
    except Exception as exc:                              # the report must not hide the tests' own result
        print(f"\nchecked build: status unavailable ({exc!r})")
        session.exitstatus = 1
        return
    print(f"\nchecked build: violations, site, index, extent = {status}")
    if status is None or status[0] != 0:
        session.exitstatus = 1
