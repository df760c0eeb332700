"""B200 configuration-sweep library: Python binding of the C ABI in include/dynamo.h.

The binding is loaded on first use, so that `paper_2408_00741_b200.build` can be imported (to compile
the shared library) before the library exists.  There is no CPU implementation behind these names:
using any of them without the built library raises ImportError.
"""
import importlib

_BINDING_NAMES = ("DYN_ECUDA", "DYN_EINVAL", "DYN_EUNSUPPORTED", "DYN_EWORKSPACE", "DYN_OK", "EXPORTS", "LIB_PATH",
                  "DynError", "HostPipeline", "Profile", "SelectOut", "Space", "dyn_bin_trace", "dyn_eval_configs",
                  "dyn_eval_select", "dyn_select", "dyn_select_workspace_bytes", "dyn_set_timing_events",
                  "dyn_workspace_bytes", "dyn_eval_select_static", "DYN_STATIC_WS_BYTES", "dyn_hier_workspace_bytes", "dyn_hier_select",
                  "MixedOut", "dyn_mixed_workspace_bytes", "dyn_mixed_tuple_count", "dyn_mixed_select",
                  "dyn_reconf_workspace_bytes", "dyn_reconf_select", "dyn_bin_tokens", "dyn_carbon",
                  "dyn_probe_fma", "dyn_probe_sweep_inner", "dyn_self_check", "dyn_debug_status", "dyn_debug_selftest", "CHECKED")
__all__ = list(_BINDING_NAMES)


def __getattr__(name):
    if name in ("build", "binding"):
        return importlib.import_module(f"{__name__}.{name}")
    if name in _BINDING_NAMES:
        binding = importlib.import_module(f"{__name__}.binding")
        for n in _BINDING_NAMES:
            globals()[n] = getattr(binding, n)
        return globals()[name]
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
