"""The checking build of the library (every computed index tested before use; a violation is recorded, never a
trap): the GPU parity suite runs once more against it in a child process, and no kernel may have recorded an index
out of range.  This is the stand-in for a memory checker, which is not available here."""
import os
import subprocess
import sys

import pytest
import torch

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(code_or_args, timeout):
    env = dict(os.environ, DYN_CHECKED="1")
    return subprocess.run([sys.executable] + code_or_args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_reporting_path_records_a_planted_index():
    """The check replaces an out-of-range index by 0 and records where it happened; the ordinary build has no checks
    and says so."""
    from paper_2408_00741_b200 import build
    build.build(check=True)
    code = (
        "import torch, paper_2408_00741_b200 as dyn\n"
        "assert dyn.CHECKED and dyn.LIB_PATH.endswith('libdynamo_check.so')\n"
        "assert dyn.dyn_debug_status() == (0, 0, 0, 0)\n"
        "out = torch.zeros(1, dtype=torch.int32, device='cuda')\n"
        "dyn.dyn_debug_selftest(out)\n"
        "v, site, index, extent = dyn.dyn_debug_status()\n"
        "assert (v, index, extent) == (1, 5, 3) and site >> 16 == 12, (v, site, index, extent)\n"
        "assert int(out.item()) == 7\n"
        "assert dyn.dyn_debug_status() == (0, 0, 0, 0)      # reading clears the record\n"
        "print('ok')\n")
    r = _run(["-c", code], 300)
    assert r.returncode == 0 and "ok" in r.stdout, r.stdout + r.stderr
    import paper_2408_00741_b200 as dyn
    if not dyn.CHECKED:
        assert dyn.dyn_debug_status() is None
        with pytest.raises(dyn.DynError):
            dyn.dyn_debug_selftest(torch.zeros(1, dtype=torch.int32, device="cuda"))


def test_gpu_suite_on_the_checking_build_records_nothing():
    if os.environ.get("DYN_CHECKED", "") not in ("", "0"):
        pytest.skip("already inside the checked run")
    r = _run(["-m", "pytest", "tests", "-m", "gpu", "-q", "-x", "-p", "no:cacheprovider",
              "--ignore", os.path.join("tests", "test_gpu_checked_build.py")], 1800)
    tail = (r.stdout + r.stderr)[-3000:]
    assert r.returncode == 0, tail
    assert "checked build: violations, site, index, extent = (0, 0, 0, 0)" in r.stdout, tail
