"""Seeded synthetic inputs: request traces, profile tables, candidate spaces, load scenarios.

This module only *makes inputs*.  It holds none of the method's arithmetic (no binning, no
interpolation, no feasibility test, no energy, no argmin) and is imported neither by the CPU
oracle nor by the CUDA library; tests and the benchmark call it and hand the same arrays to both.

Shapes follow the paper: a trace record is (timestamp, input tokens, output tokens) (Sec. 3);
request classes are the 3x3 length buckets of the thresholds table (Sec. 3.1); profiles are
functions of (load, request class, TP degree, GPU frequency) sampled at a few load levels
(Sec. 4.1).  The measured H100 profiles and the production traces are not available, so the
closed forms and distributions below stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

F_MAX_MHZ = 1980.0
IN_EDGES = np.array([256, 1024], dtype=np.uint32)      # thresholds table: S <256, M <1024, L above
OUT_EDGES = np.array([100, 350], dtype=np.uint32)      # S <100, M <350, L >=350
IN_REP = np.array([128.0, 512.0, 2048.0])              # representative lengths per bucket
OUT_REP = np.array([50.0, 200.0, 600.0])
PAPER_SLO_TTFT_S = np.array([0.25, 0.40, 2.0])         # thresholds table, by input bucket
PAPER_SLO_TBT_S = 0.1
TOKEN_MAX = 8192


# --------------------------------------------------------------------------------------
# traces
# --------------------------------------------------------------------------------------
@dataclass
class TraceSpec:
    n_req: int
    duration_s: float
    window_ms: int
    seed: int
    arrival: str = "uniform"            # "uniform" | "diurnal" | "weekly"
    amplitude: float = 0.5              # diurnal sinusoid amplitude (peak/trough = (1+A)/(1-A))
    weekend_factor: float = 0.6         # weekly: days 5 and 6 of each week scaled by this
    in_median: float = 600.0
    in_sigma: float = 1.0
    out_median: float = 200.0
    out_sigma: float = 0.8

    @property
    def n_windows(self) -> int:
        return int(round(self.duration_s * 1000.0 / self.window_ms))


def _intensity(spec: TraceSpec, t_s: np.ndarray) -> np.ndarray:
    if spec.arrival == "uniform":
        return np.ones_like(t_s)
    lam = 1.0 + spec.amplitude * np.sin(2.0 * np.pi * (t_s / 86400.0 - 0.25))
    if spec.arrival == "weekly":
        day = np.floor(t_s / 86400.0).astype(np.int64) % 7
        lam = lam * np.where(day >= 5, spec.weekend_factor, 1.0)
    elif spec.arrival != "diurnal":
        raise ValueError(f"unknown arrival pattern {spec.arrival!r}")
    return lam


def make_trace(spec: TraceSpec):
    """Return (t_ms, in_tok, out_tok), each uint32[n_req], sorted by time.

    Conditional on the request count, arrivals are i.i.d. draws from the normalised rate curve
    (inverse CDF on a 1-second grid, linear inside a second), sorted and floored to milliseconds.
    Token counts are lognormal, rounded to nearest and clipped to [1, 8192].
    """
    rng = np.random.default_rng(spec.seed)
    n = int(spec.n_req)
    if spec.arrival == "uniform":
        t = rng.random(n) * spec.duration_s
    else:
        grid = np.arange(0.0, spec.duration_s + 1.0, 1.0)
        mid = 0.5 * (grid[:-1] + grid[1:])
        cdf = np.concatenate([[0.0], np.cumsum(_intensity(spec, mid))])
        cdf /= cdf[-1]
        t = np.interp(rng.random(n), cdf, grid)
    t.sort()
    t_ms = np.minimum(np.floor(t * 1000.0), spec.duration_s * 1000.0 - 1.0).astype(np.uint32)
    tin = np.exp(np.log(spec.in_median) + spec.in_sigma * rng.standard_normal(n))
    tout = np.exp(np.log(spec.out_median) + spec.out_sigma * rng.standard_normal(n))
    in_tok = np.clip(np.rint(tin), 1, TOKEN_MAX).astype(np.uint32)
    out_tok = np.clip(np.rint(tout), 1, TOKEN_MAX).astype(np.uint32)
    return t_ms, in_tok, out_tok


# --------------------------------------------------------------------------------------
# profile tables
# --------------------------------------------------------------------------------------
@dataclass
class Coefficients:
    """Per-class coefficients of the synthetic profile closed forms (after jitter)."""
    a: np.ndarray        # s per input token (TTFT)
    b: np.ndarray        # s (TBT at TP1, f_max, zero load)
    c: np.ndarray        # s per (request/s per instance)
    kappa: np.ndarray    # request/s per instance at TP1, f_max
    k: np.ndarray        # W dynamic power per GPU at f_max, full utilisation
    p_idle: np.ndarray   # W per GPU
    in_rep: np.ndarray
    out_rep: np.ndarray


@dataclass
class Profile:
    """Profile tables as the library takes them (all float32, C-contiguous)."""
    tp: np.ndarray              # int32 [T] ascending
    f_grid_mhz: np.ndarray      # float32 [R] ascending
    ttft: np.ndarray            # [C][T][R] s
    cap: np.ndarray             # [C][T][R] request/s per instance
    tbt: np.ndarray             # [C][T][R][M] s at utilisation knots m/(M-1)
    pow: np.ndarray             # [C][T][R][M] W per instance
    coef: Coefficients = field(repr=False, default=None)

    @property
    def C(self): return self.ttft.shape[0]
    @property
    def T(self): return self.ttft.shape[1]
    @property
    def R(self): return self.ttft.shape[2]
    @property
    def M(self): return self.tbt.shape[3]


def class_coefficients(jitter_seed=None, jitter=0.1) -> Coefficients:
    """Nine classes, class index = 3*input bucket + output bucket.  With a seed, each of
    (a, b, c, kappa, k, p_idle) is scaled by 1 + jitter*(2U-1), U drawn in that order, class-major."""
    C = 9
    in_rep = np.repeat(IN_REP, 3)
    out_rep = np.tile(OUT_REP, 3)
    tok = in_rep + out_rep
    a = np.full(C, 4.0e-4)
    b = np.full(C, 0.107)
    c = 0.04 * tok / 800.0
    kappa = 1.0 * 800.0 / tok
    k = np.full(C, 600.0)
    p_idle = np.full(C, 100.0)
    if jitter_seed is not None:
        u = np.random.default_rng([int(jitter_seed), 7]).random((C, 6))
        m = 1.0 + jitter * (2.0 * u - 1.0)
        a, b, c, kappa, k, p_idle = (a * m[:, 0], b * m[:, 1], c * m[:, 2],
                                     kappa * m[:, 3], k * m[:, 4], p_idle * m[:, 5])
    return Coefficients(a, b, c, kappa, k, p_idle, in_rep, out_rep)


def make_profile(tp, f_grid_mhz, M, coef: Coefficients) -> Profile:
    """Tabulate the closed forms at (f_grid[r], u_m = m/(M-1)) in fp64 and round once to fp32.

    With s = f/1980:  TTFT = a*in/(TP^0.8 s^0.9);  cap = kappa*TP^0.7*s^0.8;
    TBT(l) = b/(TP^0.7 s^0.8) + c*l;  P(u) = P_idle*TP + k*TP*s^3*u;  knot m holds l = u_m*cap.
    """
    tp = np.asarray(tp, dtype=np.int32)
    fg = np.asarray(f_grid_mhz, dtype=np.float32)
    s = fg.astype(np.float64)[None, None, :] / F_MAX_MHZ                   # [1][1][R]
    tpf = tp.astype(np.float64)[None, :, None]                              # [1][T][1]
    cc = lambda v: np.asarray(v, dtype=np.float64)[:, None, None]           # [C][1][1]
    ttft = cc(coef.a) * cc(coef.in_rep) / (tpf ** 0.8 * s ** 0.9)
    cap = cc(coef.kappa) * tpf ** 0.7 * s ** 0.8
    u = (np.arange(M, dtype=np.float64) / (M - 1))[None, None, None, :]
    load = u * cap[..., None]
    tbt = (cc(coef.b) / (tpf ** 0.7 * s ** 0.8))[..., None] + cc(coef.c)[..., None] * load
    pw = (cc(coef.p_idle) * tpf + 0.0 * s)[..., None] + (cc(coef.k) * tpf * s ** 3)[..., None] * u
    f32 = lambda x: np.ascontiguousarray(x, dtype=np.float32)
    return Profile(tp, fg, f32(ttft), f32(cap), f32(tbt), f32(pw), coef)


# --------------------------------------------------------------------------------------
# candidate space
# --------------------------------------------------------------------------------------
@dataclass
class Space:
    f_cand_mhz: np.ndarray      # float32 [F] ascending, inside the table grid
    n_max: int
    slo_ttft_s: np.ndarray      # float32 [C]
    slo_tbt_s: np.ndarray       # float32 [C]
    gpu_budget: int             # <= 0: none
    window_s: float

    @property
    def F(self): return len(self.f_cand_mhz)


def freqs_step200():
    return np.array([800, 1000, 1200, 1400, 1600, 1800, 1980], dtype=np.float32)


def freqs_8():
    return np.array([round(800 + 1180 * i / 7) for i in range(8)], dtype=np.float32)


def make_space(f_cand, n_max, window_s, C=9, slo_ttft=1.0, slo_tbt=0.1, gpu_budget=0) -> Space:
    st = np.broadcast_to(np.asarray(slo_ttft, dtype=np.float32), (C,)).copy()
    sb = np.broadcast_to(np.asarray(slo_tbt, dtype=np.float32), (C,)).copy()
    return Space(np.asarray(f_cand, dtype=np.float32), int(n_max), st, sb, int(gpu_budget),
                 float(window_s))


def paper_slos():
    """Per-class SLOs of the thresholds table (TTFT by input bucket, TBT 100 ms)."""
    return np.repeat(PAPER_SLO_TTFT_S, 3).astype(np.float32), np.full(9, PAPER_SLO_TBT_S, np.float32)


# --------------------------------------------------------------------------------------
# load scenarios
# --------------------------------------------------------------------------------------
def resample_counts(base_counts: np.ndarray, S: int, seed: int, s_begin: int = 0) -> np.ndarray:
    """Scenarios s_begin..s_begin+S-1 of per-bin counts: scenario 0 is the base itself, scenario
    s > 0 draws Poisson(base) per bin from a generator seeded (seed, s).  uint32 [S][W][C]."""
    base = np.asarray(base_counts)
    out = np.empty((S,) + base.shape, dtype=np.uint32)
    lam = base.astype(np.float64)
    for i in range(S):
        s = s_begin + i
        if s == 0:
            out[i] = base
        else:
            out[i] = np.random.default_rng([int(seed), int(s)]).poisson(lam).astype(np.uint32)
    return out


def random_loads(shape, seed, mean=2.0, zero_frac=0.05) -> np.ndarray:
    """Free-form float32 loads (gamma-distributed, some exact zeros) for kernel tests that do not
    start from a trace."""
    rng = np.random.default_rng([int(seed), 11])
    x = rng.gamma(2.0, mean / 2.0, size=shape)
    x[rng.random(size=shape) < zero_frac] = 0.0
    return x.astype(np.float32)


# --------------------------------------------------------------------------------------
# the five benchmark configurations
# --------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    trace: TraceSpec
    tp: tuple
    f_grid_mhz: np.ndarray
    f_cand_mhz: np.ndarray
    M: int
    n_max: int
    jitter_seed: object
    S: int = 1
    scenario_seed: int = 4

    @property
    def window_s(self): return self.trace.window_ms / 1000.0
    @property
    def J(self): return self.n_max * len(self.tp) * len(self.f_cand_mhz)

    def profile(self) -> Profile:
        return make_profile(self.tp, self.f_grid_mhz, self.M, class_coefficients(self.jitter_seed))

    def space(self) -> Space:
        return make_space(self.f_cand_mhz, self.n_max, self.window_s)


def workload(name: str, scale: float = 1.0) -> Workload:
    """cfg1 .. cfg5 (cfg3 has two mixes: cfg3 = conversation-like, cfg3code = code-like).
    `scale` < 1 shrinks request count and duration together (same rates, fewer windows)."""
    day, week = 86400.0, 604800.0
    f7, f8 = freqs_step200(), freqs_8()
    if name == "cfg1":
        tr = TraceSpec(20_000, 3600.0, 60_000, seed=0, arrival="uniform")
        wl = Workload(name, tr, (2, 4, 8), f7, f7, 8, 16, None)
    elif name in ("cfg2", "cfg4"):
        tr = TraceSpec(2_000_000, day, 60_000, seed=1, arrival="diurnal", amplitude=0.5)
        wl = Workload(name, tr, (1, 2, 4, 8), f8, f8, 8, 64, 1, S=4096 if name == "cfg4" else 1)
    elif name == "cfg3":
        tr = TraceSpec(14_000_000, week, 5_000, seed=2, arrival="weekly", amplitude=0.5,
                       weekend_factor=0.6, in_median=1000.0, out_median=250.0)
        wl = Workload(name, tr, (1, 2, 4, 8), f8, f8, 8, 32, 2)
    elif name == "cfg3code":
        tr = TraceSpec(14_000_000, week, 5_000, seed=3, arrival="weekly", amplitude=0.9,
                       weekend_factor=0.2, in_median=2000.0, out_median=30.0)
        wl = Workload(name, tr, (1, 2, 4, 8), f8, f8, 8, 32, 3)
    elif name == "cfg5":
        tr = TraceSpec(2_000_000, day, 60_000, seed=5, arrival="diurnal", amplitude=0.5)
        grid = (800.0 + np.arange(79) * (1180.0 / 78.0)).astype(np.float32)
        cand = (800.0 + 15.0 * np.arange(79)).astype(np.float32)
        wl = Workload(name, tr, (1, 2, 4, 8), grid, cand, 64, 256, 5)
    else:
        raise ValueError(f"unknown workload {name!r}")
    if scale != 1.0:
        n_w = max(1, int(round(wl.trace.n_windows * scale)))
        wl.trace.duration_s = n_w * wl.trace.window_ms / 1000.0
        wl.trace.n_req = max(1, int(round(wl.trace.n_req * scale)))
    return wl
