"""Pins for the oracle's hierarchical selection (Sec. 4.2: scale-out/in, shard-up/down, scale-up/down)."""
import math

import numpy as np
import pytest

import gen
import oracle


def _setup(name="cfg2", W=24, S=2, seed=3, mean=2.5, n_max=None):
    wl = gen.workload(name)
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, n_max or wl.n_max, wl.window_s)
    load = gen.random_loads((S, W, 9), seed=seed, mean=mean)
    return wl, prof, sp, load


def test_max_load_closed_form_of_the_synthetic_profile():
    """ML = min(cap, (slo - b/(TP^.7 s^.8)) / c) at the largest TP and the highest frequency (s = 1)."""
    wl, prof, sp, load = _setup("cfg1")
    r = oracle.hier_select(prof, sp, 6, 2, load)
    co = prof.coef
    tp = float(prof.tp[-1])
    for c in range(9):
        cap = co.kappa[c] * tp ** 0.7
        head = 0.1 - co.b[c] / tp ** 0.7
        expect = 0.0 if head < 0 else min(cap, head / co.c[c])
        assert r["max_load"][c] == pytest.approx(expect, rel=2e-6)
        assert expect > 0


def test_nodes_are_the_ceiling_of_peak_over_max_load():
    wl, prof, sp, load = _setup("cfg2", W=30, S=2, mean=12.0)
    load[0, :10, 0] = 0.0                                   # an idle pool still keeps one node
    e1, e2 = 10, 5
    r = oracle.hier_select(prof, sp, e1, e2, load)
    for s in range(2):
        for k1 in range(3):
            peak = load[s, k1 * e1:(k1 + 1) * e1].max(axis=0).astype(np.float64)
            for c in range(9):
                ml = r["max_load"][c]
                assert r["nodes"][s, k1, c] == max(1, math.ceil(peak[c] / ml))
    assert r["nodes"].max() >= 2 and r["nodes"].min() == 1


def test_each_level_is_the_argmin_of_its_own_restricted_problem():
    """Sharding = argmin over (n, TP) at the highest frequency and the shard epoch's peak within the node
    budget; frequency = argmin over f for that sharding at the window's load (brute force on eval_tile)."""
    wl, prof, sp, load = _setup("cfg1", W=12, S=1, mean=4.0)
    e1, e2 = 6, 3
    r = oracle.hier_select(prof, sp, e1, e2, load)
    T, F, N = prof.T, sp.F, sp.n_max
    gpn = int(prof.tp[-1])
    for k2 in range(4):
        k1 = (k2 * e2) // e1
        for c in range(9):
            budget = int(r["nodes"][0, k1, c]) * gpn
            peak = float(load[0, k2 * e2:(k2 + 1) * e2, c].max())
            E = oracle.eval_tile(prof, sp, c, peak).reshape(N, T, F)[:, :, F - 1].copy()
            for n in range(1, N + 1):
                for t in range(T):
                    if n * int(prof.tp[t]) > budget:
                        E[n - 1, t] = np.inf
            j = int(np.argmin(E.ravel()))
            expect = j if np.isfinite(E.ravel()[j]) else -1
            assert r["shard"][0, k2, c] == expect
            for w in range(k2 * e2, (k2 + 1) * e2):
                if expect < 0:
                    assert r["best_idx"][0, w, c] == -1
                    continue
                Ew = oracle.eval_tile(prof, sp, c, float(load[0, w, c])).reshape(N * T, F)[expect]
                q = int(np.argmin(Ew))
                if np.isfinite(Ew[q]):
                    assert r["best_idx"][0, w, c] == expect * F + q
                    assert r["best_E"][0, w, c] == pytest.approx(Ew[q], rel=1e-14)
                else:
                    assert r["best_idx"][0, w, c] == -1


def test_hierarchy_never_beats_the_joint_optimum_and_uses_more_energy_at_coarser_epochs():
    wl, prof, sp, load = _setup("cfg2", W=48, S=2, mean=3.0)
    joint = oracle.eval_select(prof, sp, load)
    tot = {}
    for e1, e2 in [(1, 1), (4, 2), (12, 4), (48, 12)]:
        r = oracle.hier_select(prof, sp, e1, e2, load)
        both = (r["best_idx"] >= 0) & (joint["best_idx"] >= 0)
        assert (r["best_E"][both] >= joint["best_E"][both] * (1 - 1e-12)).all()
        assert ((r["best_idx"] >= 0) <= (joint["best_idx"] >= 0)).all()     # feasible here => feasible jointly
        tot[(e1, e2)] = r["best_E"][both].sum() / joint["best_E"][both].sum()
    assert 1.0 <= tot[(1, 1)] <= tot[(48, 12)]
    assert tot[(48, 12)] > 1.0


def test_invalid_epochs_are_rejected():
    wl, prof, sp, load = _setup("cfg1", W=4, S=1)
    with pytest.raises(ValueError):
        oracle.hier_select(prof, sp, 5, 2, load)
    with pytest.raises(ValueError):
        oracle.hier_select(prof, sp, 0, 1, load)
