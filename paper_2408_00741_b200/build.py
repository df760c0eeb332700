"""Build libdynamo.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(CSRC, "libdynamo.so")
LIB_CHECK = os.path.join(CSRC, "libdynamo_check.so")      # the same sources with -DDYN_CHECK (index checks)
SOURCES = ["abi.cu", "bin_trace.cu", "resolve.cu", "sweep.cu", "select.cu", "pipeline.cu", "static_ws.cu", "hier.cu", "mixed.cu", "reconf.cu", "tokens.cu", "probe.cu"]
HEADERS = [os.path.join(CSRC, "dyn_internal.cuh"), os.path.join(CSRC, "eval_dev.cuh"), os.path.join(CSRC, "check.cuh"),
           os.path.join(ROOT, "include", "dynamo.h")]


def nvcc_command(verbose_ptxas: bool = False, check: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "--threads", "0", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    if check:
        cmd += ["-DDYN_CHECK"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB_CHECK if check else LIB]
    # the sweep's table addresses are subnormal floats: flush-to-zero arithmetic would break them silently
    assert not any(f.startswith("-ftz") or f in ("--use_fast_math", "-use_fast_math") for f in cmd)
    return cmd


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose_ptxas: bool = False, check: bool = False) -> str:
    """Builds the library (check=True: the checking build, libdynamo_check.so) if it is older than its sources."""
    lib = LIB_CHECK if check else LIB
    if force or needs_build(lib):
        subprocess.run(nvcc_command(verbose_ptxas, check), check=True, cwd=CSRC)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose_ptxas="-v" in sys.argv, check="--check" in sys.argv))
