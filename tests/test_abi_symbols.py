"""The C-ABI library loads without a GPU and exports every function include/dynamo.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "dynamo.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(dyn_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_function():
    from paper_2408_00741_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"dyn_bin_trace", "dyn_eval_configs", "dyn_select", "dyn_eval_select", "dyn_workspace_bytes",
            "dyn_strerror"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_host_side_contract_without_a_gpu():
    import paper_2408_00741_b200 as dyn
    assert set(dyn.EXPORTS) == set(_declared())
    lib = ctypes.CDLL(dyn.LIB_PATH)
    lib.dyn_strerror.restype = ctypes.c_char_p
    assert lib.dyn_strerror(0) == b"success"
    assert b"workspace" in lib.dyn_strerror(-4)
    assert lib.dyn_last_cuda_error() == 0
    # workspace sizes are pure host arithmetic
    assert dyn.dyn_select_workspace_bytes(4, 1440, 2048) % 256 == 0
    assert dyn.dyn_select_workspace_bytes(4, 1440, 2048) >= 2 * 2048 * 4 + 4 * 12
    assert dyn.dyn_select_workspace_bytes(-1, 1, 1) == 0
    # NULL arguments are rejected on the host before any CUDA call
    lib.dyn_bin_trace.restype = ctypes.c_int
    assert lib.dyn_bin_trace(None, None, None, None, ctypes.c_uint64(0), None, None, None, None) == dyn.DYN_EINVAL
    lib.dyn_eval_select.restype = ctypes.c_int
    assert lib.dyn_eval_select(None, None, None, ctypes.c_int64(1), ctypes.c_int64(1), None, None,
                               ctypes.c_size_t(0), None) == dyn.DYN_EINVAL


def test_build_keeps_subnormal_arithmetic():
    """The sweep forms table addresses as subnormal floats: the build must not ask for flush-to-zero arithmetic."""
    from paper_2408_00741_b200 import build
    cmd = build.nvcc_command()
    assert not any(f.startswith("-ftz") or "fast_math" in f for f in cmd)
    assert "arch=compute_100a,code=sm_100a" in cmd
