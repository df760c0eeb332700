"""B200 configuration-sweep library: Python binding of the C ABI in include/dynamo.h."""
from .binding import (DYN_ECUDA, DYN_EINVAL, DYN_EUNSUPPORTED, DYN_EWORKSPACE, DYN_OK, EXPORTS, LIB_PATH, DynError,  # noqa: F401
                      HostPipeline, Profile, SelectOut, Space, dyn_bin_trace, dyn_eval_configs, dyn_eval_select, dyn_select,
                      dyn_select_workspace_bytes, dyn_set_timing_events, dyn_workspace_bytes)
