"""ctypes binding of libdynamo.so: same names as the C ABI, argument marshalling only.

Device buffers are torch CUDA tensors (torch is used for device memory and streams, nothing else);
host-side descriptors (class edges, TP list, frequency grids, SLOs) are numpy arrays.  Every call
enqueues on torch's current stream and returns without synchronising.  There is no CPU path: if the
shared library has not been built the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DYN_CHECKED=1 in the environment selects the checking build of the library (index checks in every kernel)
CHECKED = os.environ.get("DYN_CHECKED", "") not in ("", "0")
LIB_PATH = os.path.join(_HERE, "csrc", "libdynamo_check.so" if CHECKED else "libdynamo.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2408_00741_b200.build` "
                      "(there is no fallback implementation)")
_lib = C.CDLL(LIB_PATH)

DYN_OK, DYN_EINVAL, DYN_ECUDA, DYN_EUNSUPPORTED, DYN_EWORKSPACE = 0, -1, -2, -3, -4
EXPORTS = ("dyn_strerror", "dyn_last_cuda_error", "dyn_bin_trace", "dyn_workspace_bytes", "dyn_eval_configs",
           "dyn_select_workspace_bytes", "dyn_select", "dyn_eval_select", "dyn_pipeline_arena_bytes",
           "dyn_pipeline_host", "dyn_set_timing_events", "dyn_eval_select_static", "dyn_hier_workspace_bytes",
           "dyn_hier_select", "dyn_mixed_workspace_bytes", "dyn_mixed_tuple_count", "dyn_mixed_select", "dyn_reconf_workspace_bytes", "dyn_reconf_select", "dyn_bin_tokens", "dyn_carbon",
           "dyn_probe_fma", "dyn_probe_sweep_inner", "dyn_self_check", "dyn_debug_status", "dyn_debug_selftest")


class DynError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.dyn_strerror(status).decode()
        if status == DYN_ECUDA:
            msg += f" [cudaError {_lib.dyn_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


class _BinSpec(C.Structure):
    _fields_ = [("window_ms", C.c_uint32), ("n_windows", C.c_uint32), ("n_in_edges", C.c_int32),
                ("n_out_edges", C.c_int32), ("in_edges", C.c_void_p), ("out_edges", C.c_void_p)]


class _Profile(C.Structure):
    _fields_ = [("C", C.c_int32), ("T", C.c_int32), ("R", C.c_int32), ("M", C.c_int32),
                ("tp", C.c_void_p), ("f_grid_mhz", C.c_void_p), ("d_ttft", C.c_void_p), ("d_cap", C.c_void_p),
                ("d_tbt", C.c_void_p), ("d_pow", C.c_void_p)]


class _Space(C.Structure):
    _fields_ = [("F", C.c_int32), ("Nmax", C.c_int32), ("f_cand_mhz", C.c_void_p), ("slo_ttft_s", C.c_void_p),
                ("slo_tbt_s", C.c_void_p), ("gpu_budget", C.c_int32), ("window_s", C.c_float)]


class _SelectOut(C.Structure):
    _fields_ = [("d_best_idx", C.c_void_p), ("d_best_E", C.c_void_p), ("d_E_total", C.c_void_p),
                ("d_n_infeasible", C.c_void_p), ("d_E_window", C.c_void_p), ("d_hist", C.c_void_p),
                ("d_gpus", C.c_void_p)]


class _ProfileHost(C.Structure):
    _fields_ = [("C", C.c_int32), ("T", C.c_int32), ("R", C.c_int32), ("M", C.c_int32),
                ("tp", C.c_void_p), ("f_grid_mhz", C.c_void_p), ("ttft", C.c_void_p), ("cap", C.c_void_p),
                ("tbt", C.c_void_p), ("pow", C.c_void_p)]


class _HostIn(C.Structure):
    _fields_ = [("t_ms", C.c_void_p), ("in_tok", C.c_void_p), ("out_tok", C.c_void_p), ("n_req", C.c_uint64),
                ("extra_load", C.c_void_p), ("S_extra", C.c_int64), ("copy_stream", C.c_void_p)]


class _HostOut(C.Structure):
    _fields_ = [("counts", C.c_void_p), ("dropped", C.c_void_p), ("best_idx", C.c_void_p), ("best_E", C.c_void_p),
                ("E_total", C.c_void_p), ("n_infeasible", C.c_void_p), ("E_window", C.c_void_p),
                ("hist", C.c_void_p), ("gpus", C.c_void_p)]


_lib.dyn_strerror.restype = C.c_char_p
_lib.dyn_strerror.argtypes = [C.c_int]
_lib.dyn_last_cuda_error.restype = C.c_int
_lib.dyn_bin_trace.restype = C.c_int
_lib.dyn_bin_trace.argtypes = [C.POINTER(_BinSpec), C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p,
                               C.c_void_p, C.c_void_p, C.c_void_p]
_lib.dyn_workspace_bytes.restype = C.c_size_t
_lib.dyn_workspace_bytes.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_int64, C.c_int64]
_lib.dyn_eval_configs.restype = C.c_int
_lib.dyn_eval_configs.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_void_p, C.c_int64, C.c_int64,
                                  C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.dyn_select_workspace_bytes.restype = C.c_size_t
_lib.dyn_select_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64]
_lib.dyn_select.restype = C.c_int
_lib.dyn_select.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                            C.POINTER(_SelectOut), C.c_void_p, C.c_size_t, C.c_void_p]
_lib.dyn_eval_select.restype = C.c_int
_lib.dyn_eval_select.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_void_p, C.c_int64, C.c_int64,
                                 C.POINTER(_SelectOut), C.c_void_p, C.c_size_t, C.c_void_p]


_lib.dyn_pipeline_arena_bytes.restype = C.c_size_t
_lib.dyn_pipeline_arena_bytes.argtypes = [C.POINTER(_BinSpec), C.POINTER(_ProfileHost), C.POINTER(_Space), C.c_uint64,
                                          C.c_int64]
_lib.dyn_pipeline_host.restype = C.c_int
_lib.dyn_pipeline_host.argtypes = [C.POINTER(_BinSpec), C.POINTER(_ProfileHost), C.POINTER(_Space), C.POINTER(_HostIn),
                                   C.POINTER(_HostOut), C.c_void_p, C.c_size_t, C.c_void_p]
_lib.dyn_set_timing_events.restype = None
_lib.dyn_set_timing_events.argtypes = [C.c_void_p, C.c_void_p]


class _HierSpec(C.Structure):
    _fields_ = [("scale_epoch_windows", C.c_int32), ("shard_epoch_windows", C.c_int32)]


_lib.dyn_hier_workspace_bytes.restype = C.c_size_t
_lib.dyn_hier_workspace_bytes.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_int64, C.c_int64]
_lib.dyn_hier_select.restype = C.c_int
_lib.dyn_hier_select.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.POINTER(_HierSpec), C.c_void_p, C.c_int64,
                                 C.c_int64, C.c_void_p, C.c_void_p, C.POINTER(_SelectOut), C.c_void_p, C.c_size_t,
                                 C.c_void_p]
_lib.dyn_eval_select_static.restype = C.c_int
_lib.dyn_eval_select_static.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_void_p, C.c_int64, C.c_int64,
                                        C.POINTER(_SelectOut), C.c_void_p]
DYN_STATIC_WS_BYTES = 4 << 20

class _MixedOut(C.Structure):
    _fields_ = [("d_counts", C.c_void_p), ("d_freq", C.c_void_p), ("d_tuple", C.c_void_p), ("d_best_E", C.c_void_p),
                ("d_E_total", C.c_void_p), ("d_n_infeasible", C.c_void_p)]


_lib.dyn_mixed_workspace_bytes.restype = C.c_size_t
_lib.dyn_mixed_workspace_bytes.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_int64, C.c_int64]
_lib.dyn_mixed_tuple_count.restype = C.c_int64
_lib.dyn_mixed_tuple_count.argtypes = [C.POINTER(_Profile), C.POINTER(_Space)]
_lib.dyn_mixed_select.restype = C.c_int
_lib.dyn_mixed_select.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_void_p, C.c_int64, C.c_int64,
                                  C.POINTER(_MixedOut), C.c_void_p, C.c_size_t, C.c_void_p]
_lib.dyn_reconf_workspace_bytes.restype = C.c_size_t
_lib.dyn_reconf_workspace_bytes.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_int64, C.c_int64]
_lib.dyn_reconf_select.restype = C.c_int
_lib.dyn_reconf_select.argtypes = [C.POINTER(_Profile), C.POINTER(_Space), C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                   C.POINTER(_SelectOut), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.dyn_bin_tokens.restype = C.c_int
_lib.dyn_bin_tokens.argtypes = [C.POINTER(_BinSpec), C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.c_void_p]
_lib.dyn_carbon.restype = C.c_int
_lib.dyn_carbon.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
_lib.dyn_debug_status.restype = C.c_int
_lib.dyn_debug_status.argtypes = [C.POINTER(C.c_uint32)] * 4
_lib.dyn_debug_selftest.restype = C.c_int
_lib.dyn_debug_selftest.argtypes = [C.c_void_p, C.c_void_p]
_lib.dyn_self_check.restype = C.c_int
_lib.dyn_self_check.argtypes = [C.c_void_p]
_lib.dyn_probe_fma.restype = C.c_int
_lib.dyn_probe_fma.argtypes = [C.c_int32, C.c_void_p, C.POINTER(C.c_double), C.c_void_p]
_lib.dyn_probe_sweep_inner.restype = C.c_int
_lib.dyn_probe_sweep_inner.argtypes = [C.c_int32, C.c_float, C.c_void_p, C.POINTER(C.c_double), C.c_void_p]


def _dev(t, dtype, what):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{what}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _host(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != DYN_OK:
        raise DynError(rc, where)


class Profile:
    """Device-resident profile tables plus their host descriptors (mirrors dyn_profile)."""

    def __init__(self, tp, f_grid_mhz, ttft, cap, tbt, pow, device="cuda"):
        self.tp = _host(tp, np.int32)
        self.f_grid_mhz = _host(f_grid_mhz, np.float32)
        as_dev = lambda x: (x if isinstance(x, torch.Tensor) else torch.from_numpy(_host(x, np.float32))).to(
            device=device, dtype=torch.float32).contiguous()
        self.d_ttft, self.d_cap, self.d_tbt, self.d_pow = as_dev(ttft), as_dev(cap), as_dev(tbt), as_dev(pow)
        self.C, self.T, self.R = self.d_ttft.shape
        self.M = self.d_tbt.shape[3]
        if (tuple(self.d_tbt.shape) != (self.C, self.T, self.R, self.M) or tuple(self.d_pow.shape) != tuple(self.d_tbt.shape)
                or tuple(self.d_cap.shape) != (self.C, self.T, self.R) or len(self.tp) != self.T
                or len(self.f_grid_mhz) != self.R):
            raise ValueError("profile tables have inconsistent shapes")

    def _struct(self):
        return _Profile(self.C, self.T, self.R, self.M, self.tp.ctypes.data, self.f_grid_mhz.ctypes.data,
                        self.d_ttft.data_ptr(), self.d_cap.data_ptr(), self.d_tbt.data_ptr(), self.d_pow.data_ptr())


class Space:
    """Candidate space and SLOs (mirrors dyn_space); host data only."""

    def __init__(self, f_cand_mhz, n_max, slo_ttft_s, slo_tbt_s, window_s, gpu_budget=0):
        self.f_cand_mhz = _host(f_cand_mhz, np.float32)
        self.n_max = int(n_max)
        self.slo_ttft_s = _host(slo_ttft_s, np.float32)
        self.slo_tbt_s = _host(slo_tbt_s, np.float32)
        self.window_s = float(window_s)
        self.gpu_budget = int(gpu_budget)

    @property
    def F(self):
        return len(self.f_cand_mhz)

    def _struct(self):
        return _Space(self.F, self.n_max, self.f_cand_mhz.ctypes.data, self.slo_ttft_s.ctypes.data,
                      self.slo_tbt_s.ctypes.data, self.gpu_budget, self.window_s)


def dyn_bin_trace(window_ms, n_windows, in_edges, out_edges, d_t_ms, d_in_tok, d_out_tok, d_counts, d_load, d_dropped,
                  n_req=None):
    """Counts (uint32 viewed as int32 tensor [W][C]), loads (float32 or None), dropped (int64 [1])."""
    ie, oe = _host(in_edges, np.uint32), _host(out_edges, np.uint32)
    spec = _BinSpec(int(window_ms), int(n_windows), len(ie), len(oe), ie.ctypes.data, oe.ctypes.data)
    n = int(d_t_ms.numel() if n_req is None else n_req)
    rc = _lib.dyn_bin_trace(C.byref(spec), _dev(d_t_ms, torch.int32, "d_t_ms"), _dev(d_in_tok, torch.int32, "d_in_tok"),
                            _dev(d_out_tok, torch.int32, "d_out_tok"), n, _dev(d_counts, torch.int32, "d_counts"),
                            _dev(d_load, torch.float32, "d_load"), _dev(d_dropped, torch.int64, "d_dropped"), _stream())
    _check(rc, "dyn_bin_trace")


def dyn_workspace_bytes(profile: Profile, space: Space, S, W) -> int:
    p, s = profile._struct(), space._struct()
    return int(_lib.dyn_workspace_bytes(C.byref(p), C.byref(s), int(S), int(W)))


def dyn_select_workspace_bytes(S, W, J) -> int:
    return int(_lib.dyn_select_workspace_bytes(int(S), int(W), int(J)))


def _ws(d_ws):
    if d_ws is None:
        return None, 0
    if not (isinstance(d_ws, torch.Tensor) and d_ws.is_cuda and d_ws.is_contiguous()):
        raise TypeError("d_ws: expected a contiguous CUDA tensor")
    return d_ws.data_ptr(), d_ws.numel() * d_ws.element_size()


def dyn_eval_configs(profile: Profile, space: Space, d_load, d_E, d_ws):
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_eval_configs(C.byref(p), C.byref(s), _dev(d_load, torch.float32, "d_load"), S, W,
                               _dev(d_E, torch.float32, "d_E"), ws, nb, _stream())
    _check(rc, "dyn_eval_configs")


class SelectOut:
    """Output buffers of the selection stage (mirrors dyn_select_out)."""

    def __init__(self, S, W, Cn, J, device="cuda", windows=True, hist=True, gpus=True):
        self.best_idx = torch.empty((S, W, Cn), dtype=torch.int32, device=device)
        self.best_E = torch.empty((S, W, Cn), dtype=torch.float32, device=device)
        self.E_total = torch.empty((S,), dtype=torch.float64, device=device)
        self.n_infeasible = torch.empty((S,), dtype=torch.int32, device=device)
        self.E_window = torch.empty((S, W), dtype=torch.float64, device=device) if windows else None
        self.hist = torch.empty((S, J), dtype=torch.int32, device=device) if hist else None
        self.gpus = torch.empty((S, W), dtype=torch.int32, device=device) if gpus else None

    def _struct(self):
        ptr = lambda t: t.data_ptr() if t is not None else None
        return _SelectOut(ptr(self.best_idx), ptr(self.best_E), ptr(self.E_total), ptr(self.n_infeasible),
                          ptr(self.E_window), ptr(self.hist), ptr(self.gpus))


def dyn_select(d_E, out: SelectOut, d_ws, n_of_j=None, tp_of_j=None):
    S, W, Cn, J = d_E.shape
    nj = _host(n_of_j, np.int32) if n_of_j is not None else None
    tj = _host(tp_of_j, np.int32) if tp_of_j is not None else None
    o = out._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_select(_dev(d_E, torch.float32, "d_E"), S, W, Cn, J, nj.ctypes.data if nj is not None else None,
                         tj.ctypes.data if tj is not None else None, C.byref(o), ws, nb, _stream())
    _check(rc, "dyn_select")


def dyn_eval_select(profile: Profile, space: Space, d_load, out: SelectOut, d_ws):
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    o = out._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_eval_select(C.byref(p), C.byref(s), _dev(d_load, torch.float32, "d_load"), S, W, C.byref(o), ws, nb,
                              _stream())
    _check(rc, "dyn_eval_select")


def dyn_set_timing_events(start=None, stop=None):
    """start/stop: torch.cuda.Event(enable_timing=True) that have been recorded once (so that their
    handles exist), or None, None to switch the instrumentation off."""
    if start is None or stop is None:
        _lib.dyn_set_timing_events(None, None)
    else:
        _lib.dyn_set_timing_events(C.c_void_p(start.cuda_event), C.c_void_p(stop.cuda_event))


class HostPipeline:
    """Marshals dyn_pipeline_host: host (CPU, ideally pinned) tensors or numpy arrays in and out, one
    caller-owned device arena.  Shapes: trace uint32 [n]; extra_load float32 [S-1][W][C] or None."""

    def __init__(self, window_ms, n_windows, in_edges, out_edges, tp, f_grid_mhz, ttft, cap, tbt, pow, space: Space):
        self.ie, self.oe = _host(in_edges, np.uint32), _host(out_edges, np.uint32)
        self.spec = _BinSpec(int(window_ms), int(n_windows), len(self.ie), len(self.oe), self.ie.ctypes.data,
                             self.oe.ctypes.data)
        self.tp, self.fg = _host(tp, np.int32), _host(f_grid_mhz, np.float32)
        self.tabs = [_host(x, np.float32) for x in (ttft, cap, tbt, pow)]
        Cn, T, R = self.tabs[0].shape
        M = self.tabs[2].shape[3]
        self.prof = _ProfileHost(Cn, T, R, M, self.tp.ctypes.data, self.fg.ctypes.data,
                                 *[t.ctypes.data for t in self.tabs])
        self.space = space
        self.W, self.Cn, self.J = int(n_windows), Cn, space.n_max * T * space.F

    def arena_bytes(self, n_req, S) -> int:
        sp = self.space._struct()
        return int(_lib.dyn_pipeline_arena_bytes(C.byref(self.spec), C.byref(self.prof), C.byref(sp), int(n_req), int(S)))

    @staticmethod
    def _hptr(x):
        if x is None:
            return None
        if isinstance(x, torch.Tensor):
            assert not x.is_cuda and x.is_contiguous()
            return x.data_ptr()
        assert x.flags["C_CONTIGUOUS"]
        return x.ctypes.data

    def run(self, t_ms, in_tok, out_tok, extra_load, out: dict, d_arena, copy_stream=None):
        """out: dict with any of counts, dropped, best_idx, best_E, E_total, n_infeasible, E_window, hist,
        gpus -> host buffers of the right size.  Enqueues on torch's current stream; synchronise before
        reading the results.  copy_stream: an optional torch.cuda.Stream on which the scenario loads are copied
        in pieces while earlier pieces are evaluated."""
        S_extra = 0 if extra_load is None else int(extra_load.shape[0])
        n = int(t_ms.shape[0])
        hin = _HostIn(self._hptr(t_ms), self._hptr(in_tok), self._hptr(out_tok), n, self._hptr(extra_load), S_extra,
                      C.c_void_p(copy_stream.cuda_stream) if copy_stream is not None else None)
        hout = _HostOut(*[self._hptr(out.get(k)) for k in ("counts", "dropped", "best_idx", "best_E", "E_total",
                                                          "n_infeasible", "E_window", "hist", "gpus")])
        sp = self.space._struct()
        ws, nb = _ws(d_arena)
        rc = _lib.dyn_pipeline_host(C.byref(self.spec), C.byref(self.prof), C.byref(sp), C.byref(hin), C.byref(hout),
                                    ws, nb, _stream())
        _check(rc, "dyn_pipeline_host")


def dyn_eval_select_static(profile: Profile, space: Space, d_load, out: SelectOut):
    """dyn_eval_select for callers that cannot allocate device memory: no workspace argument, the
    scratch is a fixed DYN_STATIC_WS_BYTES array inside the library.  Larger problems raise DynError with
    status DYN_EUNSUPPORTED.  Calls whose GPU work overlaps share that array and must be serialised."""
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    o = out._struct()
    rc = _lib.dyn_eval_select_static(C.byref(p), C.byref(s), _dev(d_load, torch.float32, "d_load"), S, W, C.byref(o),
                                     _stream())
    _check(rc, "dyn_eval_select_static")


def dyn_hier_workspace_bytes(profile: Profile, space: Space, S, W) -> int:
    p, s = profile._struct(), space._struct()
    return int(_lib.dyn_hier_workspace_bytes(C.byref(p), C.byref(s), int(S), int(W)))


def dyn_hier_select(profile: Profile, space: Space, scale_epoch_windows, shard_epoch_windows, d_load, d_nodes, d_shard,
                    out: SelectOut, d_ws):
    """Hierarchical selection: d_nodes int32 [S][K1][C], d_shard int32 [S][K2][C], per-window choice in `out`."""
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    h = _HierSpec(int(scale_epoch_windows), int(shard_epoch_windows))
    o = out._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_hier_select(C.byref(p), C.byref(s), C.byref(h), _dev(d_load, torch.float32, "d_load"), S, W,
                              _dev(d_nodes, torch.int32, "d_nodes"), _dev(d_shard, torch.int32, "d_shard"), C.byref(o),
                              ws, nb, _stream())
    _check(rc, "dyn_hier_select")


class MixedOut:
    """Output buffers of dyn_mixed_select (mirrors dyn_mixed_out)."""

    def __init__(self, S, W, Cn, T, device="cuda"):
        self.counts = torch.empty((S, W, Cn, T), dtype=torch.int32, device=device)
        self.freq = torch.empty((S, W, Cn, T), dtype=torch.int32, device=device)
        self.tuple = torch.empty((S, W, Cn), dtype=torch.int32, device=device)
        self.best_E = torch.empty((S, W, Cn), dtype=torch.float32, device=device)
        self.E_total = torch.empty((S,), dtype=torch.float64, device=device)
        self.n_infeasible = torch.empty((S,), dtype=torch.int32, device=device)

    def _struct(self):
        return _MixedOut(self.counts.data_ptr(), self.freq.data_ptr(), self.tuple.data_ptr(), self.best_E.data_ptr(),
                         self.E_total.data_ptr(), self.n_infeasible.data_ptr())


def dyn_mixed_workspace_bytes(profile: Profile, space: Space, S, W) -> int:
    p, s = profile._struct(), space._struct()
    return int(_lib.dyn_mixed_workspace_bytes(C.byref(p), C.byref(s), int(S), int(W)))


def dyn_mixed_tuple_count(profile: Profile, space: Space) -> int:
    p, s = profile._struct(), space._struct()
    return int(_lib.dyn_mixed_tuple_count(C.byref(p), C.byref(s)))


def dyn_mixed_select(profile: Profile, space: Space, d_load, out: MixedOut, d_ws):
    """Pools that mix tensor parallelisms under space.gpu_budget (> 0): per tile the count tuple of least energy."""
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    o = out._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_mixed_select(C.byref(p), C.byref(s), _dev(d_load, torch.float32, "d_load"), S, W, C.byref(o), ws, nb,
                               _stream())
    _check(rc, "dyn_mixed_select")


def dyn_reconf_workspace_bytes(profile: Profile, space: Space, S, W) -> int:
    p, s = profile._struct(), space._struct()
    return int(_lib.dyn_reconf_workspace_bytes(C.byref(p), C.byref(s), int(S), int(W)))


def dyn_reconf_select(profile: Profile, space: Space, d_R, d_load, out: SelectOut, d_path_total, d_ws):
    """Selection with re-configuration costs: d_R float32 [NS][NS] (Wh), d_path_total float64 [S][C]."""
    S, W, Cn = d_load.shape
    p, s = profile._struct(), space._struct()
    o = out._struct()
    ws, nb = _ws(d_ws)
    rc = _lib.dyn_reconf_select(C.byref(p), C.byref(s), _dev(d_R, torch.float32, "d_R"), _dev(d_load, torch.float32, "d_load"),
                                S, W, C.byref(o), _dev(d_path_total, torch.float64, "d_path_total"), ws, nb, _stream())
    _check(rc, "dyn_reconf_select")


def dyn_bin_tokens(window_ms, n_windows, in_edges, out_edges, d_t_ms, d_in_tok, d_out_tok, d_tok_in, d_tok_out,
                   d_load_tps=None, n_req=None):
    """Token sums per (window, class): d_tok_in / d_tok_out int64 tensors [W][C] (uint64 bits), d_load_tps float32 or None."""
    ie, oe = _host(in_edges, np.uint32), _host(out_edges, np.uint32)
    spec = _BinSpec(int(window_ms), int(n_windows), len(ie), len(oe), ie.ctypes.data, oe.ctypes.data)
    n = int(d_t_ms.numel() if n_req is None else n_req)
    rc = _lib.dyn_bin_tokens(C.byref(spec), _dev(d_t_ms, torch.int32, "d_t_ms"), _dev(d_in_tok, torch.int32, "d_in_tok"),
                             _dev(d_out_tok, torch.int32, "d_out_tok"), n, _dev(d_tok_in, torch.int64, "d_tok_in"),
                             _dev(d_tok_out, torch.int64, "d_tok_out"), _dev(d_load_tps, torch.float32, "d_load_tps"),
                             _stream())
    _check(rc, "dyn_bin_tokens")


def dyn_carbon(d_E_window, d_intensity, d_carbon):
    """gCO2 per scenario from window energies (float64 [S][W], Wh) and an intensity trace (float32 [W], gCO2/kWh)."""
    S, W = d_E_window.shape
    rc = _lib.dyn_carbon(_dev(d_E_window, torch.float64, "d_E_window"), _dev(d_intensity, torch.float32, "d_intensity"), S, W,
                         _dev(d_carbon, torch.float64, "d_carbon"), _stream())
    _check(rc, "dyn_carbon")


def dyn_probe_fma(iters, d_sink) -> float:
    """Enqueues the multiply-add probe; returns the fp32 operations it executes (d_sink: float32 [1])."""
    work = C.c_double(0.0)
    _check(_lib.dyn_probe_fma(int(iters), _dev(d_sink, torch.float32, "d_sink"), C.byref(work), _stream()), "dyn_probe_fma")
    return work.value


def dyn_probe_sweep_inner(iters, feasible_share, d_sink) -> float:
    """Enqueues the inner-loop probe of the sweep with the given share of feasible candidates; returns the
    candidates it evaluates (d_sink: float32 [1])."""
    work = C.c_double(0.0)
    _check(_lib.dyn_probe_sweep_inner(int(iters), float(feasible_share), _dev(d_sink, torch.float32, "d_sink"),
                                      C.byref(work), _stream()),
           "dyn_probe_sweep_inner")
    return work.value


def dyn_self_check():
    """Start-up self-check of the subnormal address arithmetic (synchronises); raises DynError with
    DYN_EUNSUPPORTED when the library was built with flush-to-zero arithmetic."""
    _check(_lib.dyn_self_check(_stream()), "dyn_self_check")


def dyn_debug_status():
    """(violations, site, index, extent) recorded by the checking build since the last call (synchronises the
    device and clears the record); None in the ordinary build, which has no checks."""
    v = [C.c_uint32(0) for _ in range(4)]
    rc = _lib.dyn_debug_status(*[C.byref(x) for x in v])
    if rc == DYN_EUNSUPPORTED:
        return None
    _check(rc, "dyn_debug_status")
    return tuple(int(x.value) for x in v)


def dyn_debug_selftest(d_out):
    """Checking build only: plants one out-of-range index behind the check (d_out: int32 [1], receives 7)."""
    _check(_lib.dyn_debug_selftest(_dev(d_out, torch.int32, "d_out"), _stream()), "dyn_debug_selftest")
