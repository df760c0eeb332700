"""Pins for the oracle's stage (b): profile lookup, feasibility (Eq. 1 constraints), energy."""
import numpy as np
import pytest
from scipy.interpolate import RegularGridInterpolator

import gen
import oracle


def _decode(j, T, F):
    return j // (T * F) + 1, (j // F) % T, j % F


def _closed_form(coef, tp, f_mhz, c, n, L, window_s, slo_ttft, slo_tbt):
    """Energy and feasibility straight from the synthetic profile formulas (no tables)."""
    s = f_mhz / gen.F_MAX_MHZ
    ttft = coef.a[c] * coef.in_rep[c] / (tp ** 0.8 * s ** 0.9)
    cap = coef.kappa[c] * tp ** 0.7 * s ** 0.8
    l = L / n
    tbt = coef.b[c] / (tp ** 0.7 * s ** 0.8) + coef.c[c] * l
    u = l / cap
    p = coef.p_idle[c] * tp + coef.k[c] * tp * s ** 3 * u
    ok = (ttft <= slo_ttft) and (tbt <= slo_tbt) and (u <= 1.0)
    return (n * p * window_s / 3600.0 if ok else np.inf), ttft, tbt, u, p


def test_worked_values_of_the_first_config():
    """Hand-checked numbers for the 1-hour configuration's constants (class MM = 4, LL = 8, SS = 0)."""
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    T, F = prof.T, sp.F
    tp = list(wl.tp)
    fr = [float(f) for f in wl.f_cand_mhz]

    def at(c, L, n, tpv, f):
        j = ((n - 1) * T + tp.index(tpv)) * F + fr.index(f)
        E, tb, pw, u, _ = oracle.eval_tile(prof, sp, c, L, details=True)
        return E[j], tb[j], pw[j], u[j]

    E, tb, pw, u = at(4, 1.5, 2, 4, 1000.0)
    assert u == pytest.approx(0.436859, rel=2e-6) and tb == pytest.approx(0.096728, rel=1e-5)
    assert pw == pytest.approx(535.069, rel=2e-6) and E == pytest.approx(17.835648, rel=2e-6)
    E, tb, _, _ = at(4, 1.5, 1, 2, 1980.0)
    assert tb == pytest.approx(0.119266, rel=1e-5) and np.isinf(E)
    E, tb, _, _ = at(8, 0.6, 3, 4, 800.0)
    assert tb == pytest.approx(0.110195, rel=1e-5) and np.isinf(E)
    E, _, _, _ = at(8, 0.6, 3, 4, 1000.0)
    assert E == pytest.approx(26.697825, rel=2e-6)
    E, _, _, _ = at(0, 0.6, 1, 2, 1400.0)
    assert E == pytest.approx(4.100003, rel=2e-6)


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_closed_form_on_grid(name):
    """On-grid frequencies: TBT and power are linear in u, so table interpolation must reproduce the
    formulas up to the fp32 rounding of the table entries."""
    wl = gen.workload(name)
    prof, sp = wl.profile(), wl.space()
    T, F = prof.T, sp.F
    rng = np.random.default_rng(5)
    for c in range(9):
        for L in [0.0, 0.37, 1.5, float(rng.random() * 6), 11.0]:
            E, tb, pw, u, _ = oracle.eval_tile(prof, sp, c, L, details=True)
            for j in rng.choice(len(E), 60, replace=False):
                n, t, q = _decode(int(j), T, F)
                Ec, ttft, tbc, uc, pc = _closed_form(prof.coef, float(prof.tp[t]), float(sp.f_cand_mhz[q]), c, n, L,
                                                     sp.window_s, 1.0, 0.1)
                assert u[j] == pytest.approx(uc, rel=3e-7, abs=1e-12)
                if uc <= 1.0:
                    assert tb[j] == pytest.approx(tbc, rel=1e-6) and pw[j] == pytest.approx(pc, rel=1e-6)
                near = abs(tbc - 0.1) < 1e-6 or abs(uc - 1) < 1e-6 or abs(ttft - 1.0) < 1e-6
                if not near:
                    if np.isinf(Ec):
                        assert np.isinf(E[j]), (c, L, n, t, q)
                    else:
                        assert E[j] == pytest.approx(Ec, rel=1e-6)


def _dyadic_problem(R=3, M=5, T=2, Cn=2, F=3, n_max=4):
    """Tables whose entries and interpolants are exact in binary: any rounding-free mistake shows."""
    tp = np.array([2, 4][:T], dtype=np.int32)
    fg = np.array([512.0, 1024.0, 2048.0][:R], dtype=np.float32)
    ttft = np.zeros((Cn, T, R), np.float32)
    cap = np.zeros((Cn, T, R), np.float32)
    tbt = np.zeros((Cn, T, R, M), np.float32)
    pw = np.zeros((Cn, T, R, M), np.float32)
    for c in range(Cn):
        for t in range(T):
            for r in range(R):
                ttft[c, t, r] = 0.5 + 0.25 * c - 0.125 * t - 0.0625 * r
                cap[c, t, r] = 2.0 + 2.0 * t + 1.0 * r + 4.0 * c
                for m in range(M):
                    tbt[c, t, r, m] = 2.0 ** -5 + m * 2.0 ** -6 * (1 + c) + t * 2.0 ** -7 - r * 2.0 ** -8
                    pw[c, t, r, m] = 64.0 * (t + 1) + 8.0 * m * (r + 1) + 16.0 * c
    prof = gen.Profile(tp, fg, ttft, cap, tbt, pw)
    sp = gen.make_space(np.array([512.0, 768.0, 2048.0][:F], np.float32), n_max, 3600.0, C=Cn,
                        slo_ttft=[0.5, 0.625][:Cn], slo_tbt=[0.0625, 0.125][:Cn])
    return prof, sp


def test_dyadic_tables_exact():
    """Bilinear value at (f = 768 halfway between rows 0 and 1, u on and between knots), exact."""
    prof, sp = _dyadic_problem()
    T, F, M = prof.T, sp.F, prof.M
    c = 1
    # candidate q=1 (768 MHz): row 0, weight 0.5.  cap = 0.5*(cap[r0]+cap[r1]).
    row, wt = oracle.resolve(prof.f_grid_mhz, sp.f_cand_mhz)
    assert row.tolist() == [0, 0, 1] and wt.tolist() == [0.0, 0.5, 1.0]
    for t in range(T):
        capq = 0.5 * (prof.cap[c, t, 0] + prof.cap[c, t, 1])
        for n in (1, 2, 4):
            for x in (0.0, 1.0, 1.5, 2.25, 4.0):                # x = u*(M-1)
                L = x / (M - 1) * capq * n
                E, tb, pw, u, _ = oracle.eval_tile(prof, sp, c, L, details=True)
                j = ((n - 1) * T + t) * F + 1
                m = min(int(np.floor(x)), M - 2)
                nu = x - m
                exp_tb = 0.5 * ((1 - nu) * prof.tbt[c, t, 0, m] + nu * prof.tbt[c, t, 0, m + 1]) + \
                         0.5 * ((1 - nu) * prof.tbt[c, t, 1, m] + nu * prof.tbt[c, t, 1, m + 1])
                exp_pw = 0.5 * ((1 - nu) * prof.pow[c, t, 0, m] + nu * prof.pow[c, t, 0, m + 1]) + \
                         0.5 * ((1 - nu) * prof.pow[c, t, 1, m] + nu * prof.pow[c, t, 1, m + 1])
                assert u[j] == pytest.approx(x / (M - 1), rel=1e-15, abs=0)
                assert tb[j] == pytest.approx(float(exp_tb), rel=1e-14)
                assert pw[j] == pytest.approx(float(exp_pw), rel=1e-14)
                ttft = 0.5 * (prof.ttft[c, t, 0] + prof.ttft[c, t, 1])
                ok = ttft <= sp.slo_ttft_s[c] and exp_tb <= sp.slo_tbt_s[c]
                assert (E[j] == pytest.approx(n * float(exp_pw) * 1.0, rel=1e-14)) if ok else np.isinf(E[j])


def test_bilinear_against_scipy_grid_interpolator():
    """Off-grid candidate frequencies (the fine-grid configuration, shrunk): the table value equals a
    library bilinear interpolation over (f, u)."""
    tp = (1, 2, 4, 8)
    grid = (800.0 + np.arange(11) * 118.0).astype(np.float32)
    cand = (800.0 + 15.0 * np.arange(0, 79, 6)).astype(np.float32)
    M = 16
    prof = gen.make_profile(tp, grid, M, gen.class_coefficients(5))
    sp = gen.make_space(cand, 6, 60.0)
    T, F = prof.T, sp.F
    u_knots = np.arange(M) / (M - 1)
    rng = np.random.default_rng(2)
    for c in (0, 4, 8):
        L = float(rng.random() * 3 + 0.2)
        E, tb, pw, u, _ = oracle.eval_tile(prof, sp, c, L, details=True)
        for t in range(T):
            f_tb = RegularGridInterpolator((grid.astype(np.float64), u_knots), prof.tbt[c, t].astype(np.float64))
            f_pw = RegularGridInterpolator((grid.astype(np.float64), u_knots), prof.pow[c, t].astype(np.float64))
            f_cap = lambda f: np.interp(f, grid.astype(np.float64), prof.cap[c, t].astype(np.float64))
            for q in range(F):
                for n in (1, 3, 6):
                    j = ((n - 1) * T + t) * F + q
                    f = float(cand[q])
                    uu = (L / n) / f_cap(f)
                    assert u[j] == pytest.approx(uu, rel=1e-13)
                    pt = [f, min(uu, 1.0)]
                    assert tb[j] == pytest.approx(float(f_tb(pt)[0]), rel=1e-12)
                    assert pw[j] == pytest.approx(float(f_pw(pt)[0]), rel=1e-12)


def test_bilinear_error_bound_against_closed_form():
    """Fine-grid configuration: off-grid power differs from the formula by at most the linear
    interpolation bound (df^2/8 * max |d2P/df2|) plus table rounding."""
    wl = gen.workload("cfg5")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, 4, 60.0)
    T, F = prof.T, sp.F
    df = 1180.0 / 78.0
    for c in (0, 5):
        L = 0.8
        E, tb, pw, u, _ = oracle.eval_tile(prof, sp, c, L, details=True)
        for t in range(T):
            tpv = float(prof.tp[t])
            for q in range(0, F, 7):
                f = float(sp.f_cand_mhz[q])
                j = ((2 - 1) * T + t) * F + q
                _, _, tbc, uc, pc = _closed_form(prof.coef, tpv, f, c, 2, L, 60.0, 1.0, 0.1)
                if uc > 1.0:
                    continue
                # P = Pidle*TP + k*TP*s^3*u with u ~ s^-0.8  =>  |d2P/df2| <= k*TP*(L/n)/kappa/TP^.7 * 2.2*1.2*s^0.2/1980^2
                bound = df * df / 8 * prof.coef.k[c] * tpv * 6.0 / gen.F_MAX_MHZ ** 2 * max(uc, 0.05) * 4 + 1e-4 * pc
                assert abs(pw[j] - pc) <= bound
                assert pw[j] == pytest.approx(pc, rel=2e-4) and tb[j] == pytest.approx(tbc, rel=2e-4)


def test_resolve_rows_and_weights():
    fg = np.array([800, 1000, 1200, 1980], dtype=np.float32)
    row, wt = oracle.resolve(fg, np.array([800, 900, 1000, 1590, 1980], dtype=np.float32))
    assert row.tolist() == [0, 0, 1, 2, 2]
    assert wt.tolist() == pytest.approx([0.0, 0.5, 0.0, 0.5, 1.0])
    with pytest.raises(ValueError):
        oracle.resolve(fg, np.array([799.0], dtype=np.float32))
    with pytest.raises(ValueError):
        oracle.resolve(fg, np.array([1981.0], dtype=np.float32))


def test_invariants_in_n():
    """Energy is non-decreasing in n at fixed (TP, f) over the feasible range; once feasible, a larger
    n stays feasible (no budget); TTFT feasibility does not depend on the load."""
    wl = gen.workload("cfg2")
    prof, sp = wl.profile(), wl.space()
    T, F, N = prof.T, sp.F, sp.n_max
    rng = np.random.default_rng(9)
    for c in range(9):
        for L in rng.random(4) * 8:
            E = oracle.eval_tile(prof, sp, c, float(L)).reshape(N, T, F)
            fin = np.isfinite(E)
            assert (fin[1:] >= fin[:-1]).all()
            with np.errstate(invalid="ignore"):
                d = E[1:] - E[:-1]
            assert (d[fin[:-1]] >= -1e-9).all()
    E0 = np.isfinite(oracle.eval_tile(prof, sp, 4, 0.0).reshape(N, T, F))
    E1 = np.isfinite(oracle.eval_tile(prof, sp, 4, 1e-6).reshape(N, T, F))
    assert (E0 == E1).all() and (E0[0] == E0[-1]).all()


def test_gpu_budget_and_slo_masks():
    wl = gen.workload("cfg1")
    prof = wl.profile()
    sp = wl.space()
    T, F, N = prof.T, sp.F, sp.n_max
    free = oracle.eval_tile(prof, sp, 4, 1.0).reshape(N, T, F)
    sp.gpu_budget = 16
    capped = oracle.eval_tile(prof, sp, 4, 1.0).reshape(N, T, F)
    for n in range(1, N + 1):
        for t in range(T):
            if n * int(prof.tp[t]) > 16:
                assert np.isinf(capped[n - 1, t]).all()
            else:
                assert (capped[n - 1, t] == free[n - 1, t]).all()
    # the paper's per-class SLOs: TTFT 250 ms for short inputs removes slow (TP, f) pairs entirely
    st, sb = gen.paper_slos()
    sp2 = gen.make_space(wl.f_cand_mhz, N, wl.window_s, slo_ttft=st, slo_tbt=sb)
    E = oracle.eval_tile(prof, sp2, 4, 0.2).reshape(N, T, F)           # class MM: TTFT SLO 0.4 s
    ttft = prof.ttft[4]                                               # [T][R], grid == candidates
    assert (np.isinf(E[:, ttft > 0.4])).all()
    assert np.isfinite(E[-1][ttft <= 0.4]).any()


def test_tensor_layout_matches_tile_calls():
    """E[s][w][c][j] of the batched call equals the single-tile call with that tile's class and load."""
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((2, 3, 9), seed=4)
    E = oracle.eval_configs(prof, sp, load)
    assert E.shape == (2, 3, 9, wl.J)
    for s, w, c in [(0, 0, 0), (1, 2, 8), (0, 1, 4), (1, 0, 5)]:
        assert np.array_equal(E[s, w, c], oracle.eval_tile(prof, sp, c, float(load[s, w, c])))
