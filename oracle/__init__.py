"""ctypes front end of the CPU oracle (oracle/dynamo_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's CPU-baseline /
reference arms, never by the CUDA package.  Builds the C file with gcc on first use (OpenMP, -O2).
Array arguments are numpy arrays; fp32 tables and loads are promoted to fp64 inside the C code.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dynamo_oracle.c")
_LIB = os.path.join(_HERE, "libdynamo_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle into oracle/libdynamo_oracle.so (rebuilds when the source is newer)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
                        "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


class _Profile(C.Structure):
    _fields_ = [("C", C.c_int32), ("T", C.c_int32), ("R", C.c_int32), ("M", C.c_int32),
                ("tp", C.c_void_p), ("f_grid", C.c_void_p), ("ttft", C.c_void_p), ("cap", C.c_void_p),
                ("tbt", C.c_void_p), ("pw", C.c_void_p)]


class _Space(C.Structure):
    _fields_ = [("F", C.c_int32), ("Nmax", C.c_int32), ("f_cand", C.c_void_p),
                ("slo_ttft", C.c_void_p), ("slo_tbt", C.c_void_p), ("gpu_budget", C.c_int32),
                ("window_s", C.c_float)]


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def set_num_threads(n: int) -> None:
    _load().orc_set_num_threads(C.c_int(int(n)))


def _p(a):
    return C.c_void_p(a.ctypes.data) if a is not None else C.c_void_p(0)


def _arr(a, dt):
    return np.ascontiguousarray(a, dtype=dt)


def bin_trace(t_ms, in_tok, out_tok, window_ms, n_windows, in_edges, out_edges):
    """Counts uint32 [W][C] and the number of requests past the last window."""
    lib = _load()
    t_ms, in_tok, out_tok = (_arr(x, np.uint32) for x in (t_ms, in_tok, out_tok))
    ie, oe = _arr(in_edges, np.uint32), _arr(out_edges, np.uint32)
    Cn = (len(ie) + 1) * (len(oe) + 1)
    counts = np.empty((int(n_windows), Cn), dtype=np.uint32)
    dropped = C.c_uint64(0)
    rc = lib.orc_bin_trace(_p(t_ms), _p(in_tok), _p(out_tok), C.c_uint64(len(t_ms)),
                           C.c_uint32(int(window_ms)), C.c_uint32(int(n_windows)),
                           _p(ie), C.c_int32(len(ie)), _p(oe), C.c_int32(len(oe)),
                           _p(counts), C.byref(dropped))
    if rc != 0:
        raise ValueError("orc_bin_trace: invalid argument")
    return counts, int(dropped.value)


def load_from_counts(counts, window_s):
    counts = _arr(counts, np.uint32)
    out = np.empty(counts.shape, dtype=np.float32)
    _load().orc_load(_p(counts), C.c_uint64(counts.size), C.c_float(float(window_s)), _p(out))
    return out


def _structs(profile, space):
    """Keep the numpy arrays alive next to the C structs that point into them."""
    keep = SimpleNamespace(
        tp=_arr(profile.tp, np.int32), fg=_arr(profile.f_grid_mhz, np.float32),
        ttft=_arr(profile.ttft, np.float32), cap=_arr(profile.cap, np.float32),
        tbt=_arr(profile.tbt, np.float32), pw=_arr(profile.pow, np.float32),
        fc=_arr(space.f_cand_mhz, np.float32), sa=_arr(space.slo_ttft_s, np.float32),
        sb=_arr(space.slo_tbt_s, np.float32))
    Cn, T, R = keep.ttft.shape
    M = keep.tbt.shape[3]
    assert keep.tbt.shape == (Cn, T, R, M) and keep.pw.shape == (Cn, T, R, M) and keep.cap.shape == (Cn, T, R)
    assert len(keep.tp) == T and len(keep.fg) == R and len(keep.sa) == Cn and len(keep.sb) == Cn
    p = _Profile(Cn, T, R, M, keep.tp.ctypes.data, keep.fg.ctypes.data, keep.ttft.ctypes.data,
                 keep.cap.ctypes.data, keep.tbt.ctypes.data, keep.pw.ctypes.data)
    s = _Space(len(keep.fc), int(space.n_max), keep.fc.ctypes.data, keep.sa.ctypes.data,
               keep.sb.ctypes.data, int(space.gpu_budget), float(space.window_s))
    return p, s, keep


def resolve(f_grid, f_cand):
    fg, fc = _arr(f_grid, np.float32), _arr(f_cand, np.float32)
    row = np.empty(len(fc), dtype=np.int32)
    wt = np.empty(len(fc), dtype=np.float64)
    rc = _load().orc_resolve(_p(fg), C.c_int32(len(fg)), _p(fc), C.c_int32(len(fc)), _p(row), _p(wt))
    if rc != 0:
        raise ValueError("orc_resolve: candidate frequency outside the table grid (or R < 2)")
    return row, wt


def eval_tile(profile, space, c, load, details=False):
    """All J energies of one tile (fp64).  With details: also TBT, power, utilisation, margin."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    row, wt = resolve(keep.fg, keep.fc)
    J = s.Nmax * p.T * s.F
    E = np.empty(J)
    if not details:
        lib.orc_eval_tile(C.byref(p), C.byref(s), _p(row), _p(wt), C.c_int32(int(c)), C.c_double(float(load)),
                          _p(E), None, None, None, None)
        return E
    tb, pw, u = np.empty(J), np.empty(J), np.empty(J)
    mg = C.c_double(0.0)
    lib.orc_eval_tile(C.byref(p), C.byref(s), _p(row), _p(wt), C.c_int32(int(c)), C.c_double(float(load)),
                      _p(E), _p(tb), _p(pw), _p(u), C.byref(mg))
    return E, tb, pw, u, float(mg.value)


def eval_configs(profile, space, load):
    """E fp64 [S][W][C][J] for loads float32 [S][W][C]."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    load = _arr(load, np.float32)
    S, W, Cn = load.shape
    assert Cn == p.C
    J = s.Nmax * p.T * s.F
    E = np.empty((S, W, Cn, J))
    rc = lib.orc_eval_configs(C.byref(p), C.byref(s), _p(load), C.c_int64(S), C.c_int64(W), _p(E))
    if rc != 0:
        raise ValueError("orc_eval_configs: invalid argument")
    return E


def select_row(E):
    E = _arr(E, np.float64)
    idx, be, e2 = C.c_int32(0), C.c_double(0.0), C.c_double(0.0)
    _load().orc_select_row(_p(E), C.c_int64(E.size), C.byref(idx), C.byref(be), C.byref(e2))
    return int(idx.value), float(be.value), float(e2.value)


def select(E):
    """Per-tile argmin of E[..., J]: (best_idx int32, best_E, E2) shaped like E without its last axis."""
    E = _arr(E, np.float64)
    J = E.shape[-1]
    tiles = E.size // J if J else 0
    idx = np.empty(E.shape[:-1], dtype=np.int32)
    be, e2 = np.empty(E.shape[:-1]), np.empty(E.shape[:-1])
    _load().orc_select(_p(E), C.c_int64(tiles), C.c_int64(J), _p(idx), _p(be), _p(e2))
    return idx, be, e2


def eval_select(profile, space, load):
    """Fused evaluate + select: dict(best_idx, best_E, E2, margin), each [S][W][C]."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    load = _arr(load, np.float32)
    S, W, Cn = load.shape
    assert Cn == p.C
    idx = np.empty((S, W, Cn), dtype=np.int32)
    be, e2, mg = np.empty((S, W, Cn)), np.empty((S, W, Cn)), np.empty((S, W, Cn))
    rc = lib.orc_eval_select(C.byref(p), C.byref(s), _p(load), C.c_int64(S), C.c_int64(W),
                             _p(idx), _p(be), _p(e2), _p(mg))
    if rc != 0:
        raise ValueError("orc_eval_select: invalid argument")
    return dict(best_idx=idx, best_E=be, E2=e2, margin=mg)


def config_tables(n_max, tp, F):
    """n_of_j and tp_of_j for j = ((n-1)*T + t)*F + q."""
    tp = np.asarray(tp, dtype=np.int32)
    T = len(tp)
    j = np.arange(int(n_max) * T * int(F))
    return (j // (T * F) + 1).astype(np.int32), tp[(j // F) % T].astype(np.int32)


def totals(best_idx, best_E, J, n_of_j=None, tp_of_j=None):
    """dict(E_total[S], n_infeasible[S], E_window[S][W], hist[S][J], gpus[S][W] or None)."""
    idx = _arr(best_idx, np.int32)
    be = _arr(best_E, np.float64)
    S, W, Cn = idx.shape
    et = np.empty(S)
    bad = np.empty(S, dtype=np.uint32)
    ew = np.empty((S, W))
    hist = np.empty((S, int(J)), dtype=np.uint32)
    have = n_of_j is not None and tp_of_j is not None
    gp = np.empty((S, W), dtype=np.uint32) if have else None
    nj = _arr(n_of_j, np.int32) if have else None
    tj = _arr(tp_of_j, np.int32) if have else None
    _load().orc_totals(_p(idx), _p(be), C.c_int64(S), C.c_int64(W), C.c_int32(Cn), C.c_int64(int(J)),
                       _p(nj), _p(tj), _p(et), _p(bad), _p(ew), _p(hist), _p(gp))
    return dict(E_total=et, n_infeasible=bad, E_window=ew, hist=hist, gpus=gp)


def hier_select(profile, space, e1, e2, load):
    """Hierarchical selection (nodes per pool -> sharding -> frequency): dict(nodes[S][K1][C],
    shard[S][K2][C], best_idx, best_E [S][W][C], max_load[C]) plus the diagnostics nodes_frac,
    shard_margin, shard_gap, freq_margin, freq_gap used for parity exemptions."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    load = _arr(load, np.float32)
    S, W, Cn = load.shape
    assert Cn == p.C
    if int(e1) < 1 or int(e2) < 1 or int(e1) % int(e2) != 0:
        raise ValueError("orc_hier_select: epochs must be >= 1 and e1 a multiple of e2")
    K1, K2 = -(-W // int(e1)), -(-W // int(e2))
    out = dict(nodes=np.empty((S, K1, Cn), np.int32), shard=np.empty((S, K2, Cn), np.int32),
               best_idx=np.empty((S, W, Cn), np.int32), best_E=np.empty((S, W, Cn)),
               max_load=np.empty(Cn), nodes_frac=np.empty((S, K1, Cn)), shard_margin=np.empty((S, K2, Cn)),
               shard_gap=np.empty((S, K2, Cn)), freq_margin=np.empty((S, W, Cn)), freq_gap=np.empty((S, W, Cn)))
    rc = lib.orc_hier_select(C.byref(p), C.byref(s), C.c_int32(int(e1)), C.c_int32(int(e2)), _p(load),
                             C.c_int64(S), C.c_int64(W), _p(out["nodes"]), _p(out["shard"]), _p(out["best_idx"]),
                             _p(out["best_E"]), _p(out["max_load"]), _p(out["nodes_frac"]), _p(out["shard_margin"]),
                             _p(out["shard_gap"]), _p(out["freq_margin"]), _p(out["freq_gap"]))
    if rc != 0:
        raise ValueError("orc_hier_select: invalid argument (epochs must be >= 1 and e1 a multiple of e2)")
    return out


def mixed_select(profile, space, load):
    """Pools that mix tensor parallelisms (Eq. 1 in full, by enumeration; needs space.gpu_budget > 0):
    dict(counts[S][W][C][T], freq[S][W][C][T], tuple_no, best_E, E2, margin [S][W][C])."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    load = _arr(load, np.float32)
    S, W, Cn = load.shape
    assert Cn == p.C
    out = dict(counts=np.empty((S, W, Cn, p.T), np.int32), freq=np.empty((S, W, Cn, p.T), np.int32),
               tuple_no=np.empty((S, W, Cn), np.int32), best_E=np.empty((S, W, Cn)), E2=np.empty((S, W, Cn)),
               margin=np.empty((S, W, Cn)))
    rc = lib.orc_mixed_select(C.byref(p), C.byref(s), _p(load), C.c_int64(S), C.c_int64(W), _p(out["counts"]),
                              _p(out["freq"]), _p(out["tuple_no"]), _p(out["best_E"]), _p(out["E2"]), _p(out["margin"]))
    if rc != 0:
        raise ValueError("orc_mixed_select: invalid argument (a GPU budget > 0 is required)")
    return out


def reconf_select(profile, space, R, load):
    """Selection with re-configuration costs: R float32 [NS][NS] (Wh, NS = n_max*T, state = (n-1)*T + t).
    dict(best_idx[S][W][C], best_E[S][W][C], path_total[S][C])."""
    lib = _load()
    p, s, keep = _structs(profile, space)
    load = _arr(load, np.float32)
    S, W, Cn = load.shape
    NS = int(space.n_max) * int(p.T)
    R = _arr(R, np.float32)
    assert R.shape == (NS, NS) and Cn == p.C
    out = dict(best_idx=np.empty((S, W, Cn), np.int32), best_E=np.empty((S, W, Cn)), path_total=np.empty((S, Cn)))
    rc = lib.orc_reconf_select(C.byref(p), C.byref(s), _p(R), _p(load), C.c_int64(S), C.c_int64(W),
                               _p(out["best_idx"]), _p(out["best_E"]), _p(out["path_total"]))
    if rc != 0:
        raise ValueError("orc_reconf_select: invalid argument")
    return out


def bin_tokens(t_ms, in_tok, out_tok, window_ms, n_windows, in_edges, out_edges):
    """Sums of input and output tokens per (window, class): (tok_in, tok_out), uint64 [W][C]."""
    t, a, b = _arr(t_ms, np.uint32), _arr(in_tok, np.uint32), _arr(out_tok, np.uint32)
    ie, oe = _arr(in_edges, np.uint32), _arr(out_edges, np.uint32)
    Cn = (len(ie) + 1) * (len(oe) + 1)
    ti = np.empty((int(n_windows), Cn), np.uint64)
    to = np.empty((int(n_windows), Cn), np.uint64)
    rc = _load().orc_bin_tokens(_p(t), _p(a), _p(b), C.c_uint64(len(t)), C.c_uint32(int(window_ms)),
                                C.c_uint32(int(n_windows)), _p(ie), C.c_int32(len(ie)), _p(oe), C.c_int32(len(oe)),
                                _p(ti), _p(to))
    if rc != 0:
        raise ValueError("orc_bin_tokens: invalid argument")
    return ti, to


def load_tps(tok_in, tok_out, window_s):
    ti, to = _arr(tok_in, np.uint64), _arr(tok_out, np.uint64)
    out = np.empty(ti.shape, np.float32)
    _load().orc_load_tps(_p(ti), _p(to), C.c_uint64(ti.size), C.c_float(float(window_s)), _p(out))
    return out


def carbon(E_window, intensity):
    """gCO2 per scenario: sum over windows of E_window [Wh] * intensity [gCO2/kWh] / 1000."""
    ew, it = _arr(E_window, np.float64), _arr(intensity, np.float32)
    S, W = ew.shape
    assert it.shape == (W,)
    out = np.empty(S, np.float64)
    _load().orc_carbon(_p(ew), _p(it), C.c_int64(S), C.c_int64(W), _p(out))
    return out
