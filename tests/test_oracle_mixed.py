"""Pins of the oracle's mixed-parallelism pools (Eq. 1 in full): an independent restatement on
numpy.interp and itertools over tiny grids, the closed form of the synthetic profile for one worked
tuple, the reduction to single-type pools, and invariants in the budget."""
import itertools

import numpy as np
import pytest

import gen
import oracle


def _interp_tables(prof, sp, c, t, q, u):
    """TTFT, cap, TBT, P of (class, TP index, candidate frequency) at utilisation u, via numpy.interp."""
    fg = prof.f_grid_mhz.astype(np.float64)
    f = float(sp.f_cand_mhz[q])
    uk = np.arange(prof.M) / (prof.M - 1)
    ttft = np.interp(f, fg, prof.ttft[c, t].astype(np.float64))
    cap = np.interp(f, fg, prof.cap[c, t].astype(np.float64))
    tb = np.interp(f, fg, [np.interp(u, uk, prof.tbt[c, t, r].astype(np.float64)) for r in range(prof.R)])
    pw = np.interp(f, fg, [np.interp(u, uk, prof.pow[c, t, r].astype(np.float64)) for r in range(prof.R)])
    return ttft, cap, tb, pw


def _brute_tile(prof, sp, c, L):
    T, F, N, B = prof.T, sp.F, sp.n_max, sp.gpu_budget
    capH = [np.interp(float(sp.f_cand_mhz[F - 1]), prof.f_grid_mhz.astype(np.float64),
                      prof.cap[c, t].astype(np.float64)) for t in range(T)]
    best = (np.inf, None, None, -1)
    number = -1
    # odometer order with n_0 fastest == itertools.product over reversed digits
    for rev in itertools.product(range(N + 1), repeat=T):
        n = rev[::-1]
        if sum(n) == 0 or sum(n[t] * int(prof.tp[t]) for t in range(T)) > B:
            continue
        number += 1
        A = sum(n[t] * capH[t] for t in range(T))
        E, qs = 0.0, []
        for t in range(T):
            if n[t] == 0:
                qs.append(-1)
                continue
            share = L * n[t] * capH[t] / A
            eg, qg = np.inf, -1
            for q in range(F):
                _, cap, _, _ = _interp_tables(prof, sp, c, t, q, 0.0)
                u = share / n[t] / cap
                ttft, _, tb, pw = _interp_tables(prof, sp, c, t, q, min(u, 1.0))
                ok = ttft <= sp.slo_ttft_s[c] and tb <= sp.slo_tbt_s[c] and u <= 1.0
                e = n[t] * pw * sp.window_s / 3600.0 if ok else np.inf
                if e < eg:
                    eg, qg = e, q
            E += eg
            qs.append(qg)
        if E < best[0]:
            best = (E, n, qs, number)
    return best


def _tiny(seed, T=2, F=3, N=3, M=3, R=4, Cn=2, budget=8):
    rng = np.random.default_rng(seed)
    tp = np.array([1, 2, 4, 8][:T], np.int32)
    fg = np.linspace(800, 1980, R).astype(np.float32)
    fc = np.sort(rng.uniform(800, 1980, F)).astype(np.float32)
    fc[-1] = 1980.0
    cap = (rng.uniform(0.5, 2.0, (Cn, T, 1)) * np.linspace(0.6, 1.0, R)[None, None, :]).astype(np.float32)
    ttft = rng.uniform(0.1, 0.6, (Cn, T, R)).astype(np.float32)
    tbt = np.sort(rng.uniform(0.02, 0.14, (Cn, T, R, M)), axis=3).astype(np.float32)
    pw = np.sort(rng.uniform(100, 900, (Cn, T, R, M)), axis=3).astype(np.float32)
    prof = gen.Profile(tp, fg, ttft, cap, tbt, pw)
    sp = gen.make_space(fc, N, 30.0, C=Cn, slo_ttft=0.5, slo_tbt=0.1, gpu_budget=budget)
    return prof, sp


@pytest.mark.parametrize("seed,T,budget", [(1, 2, 5), (2, 2, 3), (3, 3, 9), (4, 3, 4)])
def test_brute_force_tiny_grids(seed, T, budget):
    prof, sp = _tiny(seed, T=T, budget=budget)
    rng = np.random.default_rng(100 + seed)
    load = rng.uniform(0.0, 4.0, (2, 3, prof.C)).astype(np.float32)
    load[0, 0, 0] = 0.0
    load[1, 2, 1] = 50.0                                   # more than any tuple carries
    r = oracle.mixed_select(prof, sp, load)
    for s in range(2):
        for w in range(3):
            for c in range(prof.C):
                E, n, qs, number = _brute_tile(prof, sp, c, float(load[s, w, c]))
                if n is None:
                    assert r["tuple_no"][s, w, c] == -1 and np.isinf(r["best_E"][s, w, c])
                    assert (r["counts"][s, w, c] == -1).all() and (r["freq"][s, w, c] == -1).all()
                    continue
                assert r["tuple_no"][s, w, c] == number
                assert tuple(r["counts"][s, w, c]) == tuple(n)
                assert list(r["freq"][s, w, c]) == qs
                assert r["best_E"][s, w, c] == pytest.approx(E, rel=1e-12)
    assert np.isinf(r["best_E"][1, 2, 1])


def test_worked_tuple_closed_form():
    """One tuple forced by the budget and the count range (one TP2 and one TP4 instance, class MM of the
    synthetic profile, on-grid frequencies): shares, feasibility and energy from the closed forms."""
    coef = gen.class_coefficients(None)
    f = gen.freqs_step200()
    prof = gen.make_profile((2, 4), f, 8, coef)
    # budget 6 with counts 0..1: tuples (1,0), (0,1), (1,1); a load only (1,1) can carry
    sp = gen.make_space(f, 1, 60.0, gpu_budget=6)
    c = 4                                                  # MM: in 512, out 200
    kappa, b, cc, k, pid = coef.kappa[c], coef.b[c], coef.c[c], coef.k[c], coef.p_idle[c]
    capH = [kappa * tp ** 0.7 for tp in (2, 4)]            # s = 1 at 1980 MHz
    L = np.float32(2.2)        # TBT caps one TP2 instance at 0.96 and one TP4 instance at 1.67 requests/s
    load = np.zeros((1, 1, 9), np.float32)
    load[0, 0, c] = L
    r = oracle.mixed_select(prof, sp, load)
    assert tuple(r["counts"][0, 0, c]) == (1, 1)
    A = capH[0] + capH[1]
    total, qs = 0.0, []
    for t, tp in enumerate((2, 4)):
        l = float(L) * capH[t] / A                         # one instance per group
        best, bq = np.inf, -1
        for q, fq in enumerate(f.astype(np.float64)):
            s = fq / 1980.0
            cap = kappa * tp ** 0.7 * s ** 0.8
            u = l / cap
            tbt = b / (tp ** 0.7 * s ** 0.8) + cc * l
            ttft = coef.a[c] * coef.in_rep[c] / (tp ** 0.8 * s ** 0.9)
            if u <= 1.0 and tbt <= 0.1 and ttft <= 1.0:
                e = (pid * tp + k * tp * s ** 3 * u) * 60.0 / 3600.0
                if e < best:
                    best, bq = e, q
        total += best
        qs.append(bq)
    assert list(r["freq"][0, 0, c]) == qs
    assert r["best_E"][0, 0, c] == pytest.approx(total, rel=2e-7)      # fp32 rounding of the table entries


def test_single_type_reduces_to_single_pool():
    """With one TP degree a tuple is an instance count and its share is the whole load: the choice is the
    single-type selection under the same GPU budget."""
    wl = gen.workload("cfg1")
    prof1 = gen.make_profile((4,), wl.f_grid_mhz, wl.M, gen.class_coefficients(3))
    sp = gen.make_space(wl.f_cand_mhz, 12, 60.0, gpu_budget=40)
    load = gen.random_loads((2, 5, 9), seed=5, mean=3.0)
    m = oracle.mixed_select(prof1, sp, load)
    r = oracle.eval_select(prof1, sp, load)
    F = sp.F
    feas = r["best_idx"] >= 0
    assert ((m["tuple_no"] >= 0) == feas).all()
    assert (m["counts"][..., 0][feas] == r["best_idx"][feas] // F + 1).all()
    assert (m["freq"][..., 0][feas] == r["best_idx"][feas] % F).all()
    np.testing.assert_allclose(m["best_E"][feas], r["best_E"][feas], rtol=1e-13)


def test_mixing_never_costs_more_and_budget_is_monotone():
    wl = gen.workload("cfg1")
    prof = wl.profile()
    load = gen.random_loads((1, 12, 9), seed=6, mean=4.0)
    prev = None
    for budget in (8, 16, 32):
        sp = gen.make_space(wl.f_cand_mhz, 6, 60.0, gpu_budget=budget)
        m = oracle.mixed_select(prof, sp, load)
        single = oracle.eval_select(prof, sp, load)
        # single-type pools are tuples with one non-zero count (share = whole load)
        assert (m["best_E"] <= single["best_E"] * (1 + 1e-12)).all()
        gp = (m["counts"] * prof.tp[None, None, None, :]).sum(axis=3)
        assert (gp[m["tuple_no"] >= 0] <= budget).all()
        assert ((m["counts"] == 0) == (m["freq"] == -1))[m["tuple_no"] >= 0].all()
        if prev is not None:
            assert (m["best_E"] <= prev * (1 + 1e-12)).all()
        prev = m["best_E"]
    assert (m["best_E"] < single["best_E"] * (1 - 1e-6)).any()       # mixing does help somewhere


def test_needs_a_budget():
    wl = gen.workload("cfg1")
    with pytest.raises(ValueError):
        oracle.mixed_select(wl.profile(), gen.make_space(wl.f_cand_mhz, 4, 60.0), np.zeros((1, 1, 9), np.float32))
