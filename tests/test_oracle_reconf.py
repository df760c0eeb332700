"""Pins of the oracle's selection with re-configuration costs (a shortest path over the windows): brute force over
all schedules on tiny cases, the two limits of the overhead table (free: the per-window selection; prohibitive:
the best fixed sharding), bounds between them, and a run on the paper's re-sharding overheads."""
import itertools
import os

import numpy as np
import pytest

import gen
import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _window_costs(prof, sp, load_sc):
    """cost[w][sigma] = least energy over the frequencies, from the (separately pinned) per-candidate energies."""
    T, F, N = prof.T, sp.F, sp.n_max
    out = []
    for (c, L) in load_sc:
        E = oracle.eval_tile(prof, sp, c, float(L))
        out.append(E.reshape(N * T, F).min(axis=1))
    return np.array(out)


def _small(seed, budget=0):
    wl = gen.workload("cfg1")
    prof = gen.make_profile((2, 4), wl.f_grid_mhz, wl.M, gen.class_coefficients(seed))
    sp = gen.make_space(wl.f_cand_mhz[[0, 3, 6]], 2, 60.0, gpu_budget=budget)
    return prof, sp


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_brute_force_over_all_schedules(seed):
    prof, sp = _small(seed)
    NS, W = sp.n_max * prof.T, 5
    rng = np.random.default_rng(seed)
    R = rng.uniform(0.0, 6.0, (NS, NS)).astype(np.float32)
    np.fill_diagonal(R, 0.0)
    load = rng.uniform(0.2, 2.5, (2, W, 9)).astype(np.float32)
    r = oracle.reconf_select(prof, sp, R, load)
    switches = 0
    for s in range(2):
        for c in (0, 4, 8):
            cost = _window_costs(prof, sp, [(c, load[s, w, c]) for w in range(W)])
            best, arg = np.inf, None
            for path in itertools.product(range(NS), repeat=W):
                v = sum(cost[w, g] for w, g in enumerate(path)) + sum(float(R[a, b]) for a, b in zip(path, path[1:]))
                if v < best:
                    best, arg = v, path
            if not np.isfinite(best):
                assert (r["best_idx"][s, :, c] == -1).all() and np.isinf(r["path_total"][s, c])
                continue
            assert r["path_total"][s, c] == pytest.approx(best, rel=1e-12)
            assert tuple(r["best_idx"][s, :, c] // sp.F) == arg
            switches += len(set(arg)) > 1
            np.testing.assert_allclose(r["best_E"][s, :, c], [cost[w, g] for w, g in enumerate(arg)], rtol=1e-12)
    assert switches >= 1                                  # some schedule does re-configure


def test_free_reconfiguration_is_the_per_window_selection():
    prof, sp = _small(4)
    NS = sp.n_max * prof.T
    load = gen.random_loads((2, 12, 9), seed=41, mean=1.2)
    r = oracle.reconf_select(prof, sp, np.zeros((NS, NS), np.float32), load)
    ref = oracle.eval_select(prof, sp, load)
    ok = np.isfinite(r["path_total"])                     # classes whose every window has a feasible candidate
    assert ok.any()
    for s, c in zip(*np.nonzero(ok)):
        assert (r["best_idx"][s, :, c] == ref["best_idx"][s, :, c]).all()
        np.testing.assert_allclose(r["best_E"][s, :, c], ref["best_E"][s, :, c], rtol=1e-13)
        assert r["path_total"][s, c] == pytest.approx(ref["best_E"][s, :, c].sum(), rel=1e-12)
    for s, c in zip(*np.nonzero(~ok)):
        assert (ref["best_idx"][s, :, c] < 0).any() and (r["best_idx"][s, :, c] == -1).all()


def test_prohibitive_reconfiguration_is_the_best_fixed_sharding_and_bounds():
    prof, sp = _small(5)
    NS, W = sp.n_max * prof.T, 10
    load = gen.random_loads((1, W, 9), seed=42, mean=1.0, zero_frac=0.0)
    wall = np.full((NS, NS), 1e9, np.float32)
    np.fill_diagonal(wall, 0.0)
    fixed = oracle.reconf_select(prof, sp, wall, load)
    free = oracle.reconf_select(prof, sp, np.zeros((NS, NS), np.float32), load)
    rng = np.random.default_rng(7)
    some = rng.uniform(0, 3, (NS, NS)).astype(np.float32)
    np.fill_diagonal(some, 0.0)
    mid = oracle.reconf_select(prof, sp, some, load)
    for c in range(9):
        cost = _window_costs(prof, sp, [(c, load[0, w, c]) for w in range(W)])
        tot = cost.sum(axis=0)
        if np.isfinite(tot).any():
            g = int(np.argmin(tot))
            assert (fixed["best_idx"][0, :, c] // sp.F == g).all()
            assert fixed["path_total"][0, c] == pytest.approx(tot[g], rel=1e-12)
        if np.isfinite(fixed["path_total"][0, c]):
            assert free["path_total"][0, c] <= mid["path_total"][0, c] * (1 + 1e-12)
            assert mid["path_total"][0, c] <= fixed["path_total"][0, c] * (1 + 1e-12)
            # the reported total is the window energies plus the transitions of the reported path
            st = mid["best_idx"][0, :, c] // sp.F
            again = mid["best_E"][0, :, c].sum() + sum(float(some[a, b]) for a, b in zip(st, st[1:]))
            assert mid["path_total"][0, c] == pytest.approx(again, rel=1e-12)


def paper_reshard_table():
    """The fixture's overheads as {(n_src, tp_src, n_dst, tp_dst): units of T}."""
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "reshard_overheads.txt")) if l.strip() and l[0] != "#"]
    names = rows[0][1:]
    tab = {}
    for r in rows[1:]:
        ns, ts = map(int, r[0].split("x"))
        for name, v in zip(names, r[1:]):
            nd, td = map(int, name.split("x"))
            tab[(ns, ts, nd, td)] = int(v)
    return tab


def test_paper_reshard_overheads_as_the_overhead_table():
    """States (n, TP) of one 8-GPU node with the paper's transfer times (T = 50 ms at 8 x 700 W), 4T where the table
    has no entry: transitions the table gives as free are taken whenever they save energy."""
    tab = paper_reshard_table()
    assert tab[(1, 2, 4, 2)] == 4 and tab[(4, 2, 1, 8)] == 0 and tab[(1, 4, 1, 8)] == 1 and tab[(1, 8, 2, 4)] == 1
    wl = gen.workload("cfg1")
    prof = wl.profile()                                    # TP 2 / 4 / 8
    sp = gen.make_space(wl.f_cand_mhz, 4, 60.0, gpu_budget=8)
    T, NS = prof.T, 4 * prof.T
    unit_wh = 0.050 * 8 * 700.0 / 3600.0                   # one T of an 8-GPU node at full power, in Wh
    R = np.full((NS, NS), 4 * unit_wh, np.float32)
    for (ns, ts, nd, td), v in tab.items():
        a = (ns - 1) * T + list(prof.tp).index(ts)
        b = (nd - 1) * T + list(prof.tp).index(td)
        R[a, b] = v * unit_wh
    np.fill_diagonal(R, 0.0)
    load = gen.random_loads((1, 30, 9), seed=43, mean=1.0, zero_frac=0.0)
    r = oracle.reconf_select(prof, sp, R, load)
    free = oracle.reconf_select(prof, sp, np.zeros((NS, NS), np.float32), load)
    ok = np.isfinite(r["path_total"][0])
    assert ok.any()
    assert (r["path_total"][0][ok] >= free["path_total"][0][ok] * (1 - 1e-12)).all()
    gp = (r["best_idx"][0] // sp.F // T + 1) * prof.tp[(r["best_idx"][0] // sp.F) % T]
    assert (gp[:, ok] <= 8).all()
