"""Pins for the oracle's stage (c): masked argmin with lowest-index tie-break, totals."""
import os

import numpy as np
import pytest

import gen
import oracle


def _paper_rows(golden_dir):
    rows = []
    for line in open(os.path.join(golden_dir, "paper_energy_tables.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tab, label, cells, col = [x.strip() for x in line.split(";")]
        E = np.array([np.inf if v == "x" else float(v) for v in cells.split()])
        assert len(E) == 12
        rows.append((tab, label, E, int(col)))
    return rows


def test_paper_tables_choose_the_bold_cell(golden_dir):
    """Tables 1-3: gray cells are infeasible, the bold cell is the minimum-energy feasible one."""
    rows = _paper_rows(golden_dir)
    assert len(rows) == 18
    for tab, label, E, col in rows:
        idx, be, e2 = oracle.select_row(E)
        assert idx == col, (tab, label)
        assert be == E[col] and e2 > be
    # statements of the text: SS -> TP2 @ 1.2 GHz, LL -> TP8 @ 1.6 GHz, low load -> TP4 @ 1.2, high -> TP4 @ 2.0
    by = {(t, l): c for t, l, _, c in rows}
    assert by[("T1", "SS")] == 1 and by[("T1", "LL")] == 10 and by[("T2", "Low")] == 5 and by[("T2", "High")] == 7
    # the lowest-power feasible column for LL (TP8 @ 1.2, col 9) is not the energy optimum
    assert by[("T1", "LL")] != 9
    # batched form over all rows at once
    idx, be, e2 = oracle.select(np.stack([r[2] for r in rows]))
    assert idx.tolist() == [r[3] for r in rows]


def test_ties_all_infeasible_and_runner_up():
    assert oracle.select_row(np.array([3.0, 1.0, 1.0, 2.0, 1.0])) == (1, 1.0, 1.0)
    idx, be, e2 = oracle.select_row(np.array([np.inf, np.inf]))
    assert idx == -1 and np.isinf(be) and np.isinf(e2)
    assert oracle.select_row(np.array([np.inf, 5.0, np.inf])) == (1, 5.0, np.inf)
    assert oracle.select_row(np.array([7.0])) == (0, 7.0, np.inf)
    assert oracle.select_row(np.array([2.0, 9.0, 4.0])) == (0, 2.0, 4.0)


def test_against_numpy_argmin():
    """numpy.argmin returns the first minimum: the same rule."""
    rng = np.random.default_rng(0)
    E = np.round(rng.random((200, 37)) * 8) / 4            # many exact duplicates
    E[rng.random(E.shape) < 0.4] = np.inf
    E[:5] = np.inf
    idx, be, e2 = oracle.select(E)
    ref = np.argmin(E, axis=1)
    ref_min = E[np.arange(len(E)), ref]
    ref = np.where(np.isinf(ref_min), -1, ref)
    assert (idx == ref).all() and (be == ref_min).all()
    for i in range(len(E)):
        others = np.delete(E[i], ref[i]) if ref[i] >= 0 else E[i]
        assert e2[i] == others.min()


def test_totals_invariants():
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((3, 20, 9), seed=1, mean=3.0)
    load[1, 4, :] = 500.0                                    # beyond any capacity: infeasible tiles
    r = oracle.eval_select(prof, sp, load)
    nj, tj = oracle.config_tables(sp.n_max, prof.tp, sp.F)
    tot = oracle.totals(r["best_idx"], r["best_E"], wl.J, nj, tj)
    assert tot["n_infeasible"].tolist() == [int((r["best_idx"][s] < 0).sum()) for s in range(3)]
    assert tot["n_infeasible"][1] >= 9
    assert np.allclose(tot["E_window"].sum(axis=1), tot["E_total"], rtol=1e-13)
    assert (tot["hist"].sum(axis=1) == 20 * 9 - tot["n_infeasible"]).all()
    assert tot["E_window"][1, 4] == 0.0 and tot["gpus"][1, 4] == 0
    fin = np.where(r["best_idx"] >= 0, r["best_E"], 0.0)
    assert np.allclose(tot["E_total"], fin.sum(axis=(1, 2)), rtol=1e-13)
    # gpus = sum over classes of n* x TP*
    idx = r["best_idx"]
    g = np.where(idx >= 0, nj[np.maximum(idx, 0)] * tj[np.maximum(idx, 0)], 0).sum(axis=2)
    assert (tot["gpus"] == g).all()
    # config tables follow j = ((n-1)*T + t)*F + q
    T, F = prof.T, sp.F
    j = ((5 - 1) * T + 2) * F + 3
    assert nj[j] == 5 and tj[j] == prof.tp[2]


def test_eval_select_equals_eval_then_select():
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((2, 7, 9), seed=8)
    fused = oracle.eval_select(prof, sp, load)
    E = oracle.eval_configs(prof, sp, load)
    idx, be, e2 = oracle.select(E)
    assert np.array_equal(fused["best_idx"], idx) and np.array_equal(fused["best_E"], be)
    assert np.array_equal(fused["E2"], e2)
