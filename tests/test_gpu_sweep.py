"""GPU parity, stages (b) and (c): energies within 1e-5 relative of the oracle, chosen index identical
outside near-ties / near-bound candidates, totals within 1e-5, histograms equal."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import (REL_TOL, check_selection, gpu_eval_select, gpu_profile_space, out_to_host, random_tables,
                    tables_with_few_rows_without_threshold)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _small(name, W, S=1, n_max=None, seed=0, budget=0, paper_slo=False):
    wl = gen.workload(name)
    prof = wl.profile()
    n_max = n_max or wl.n_max
    if paper_slo:
        st, sb = gen.paper_slos()
        sp = gen.make_space(wl.f_cand_mhz, n_max, wl.window_s, slo_ttft=st, slo_tbt=sb, gpu_budget=budget)
    else:
        sp = gen.make_space(wl.f_cand_mhz, n_max, wl.window_s, gpu_budget=budget)
    load = gen.random_loads((S, W, 9), seed=seed, mean=2.5)
    load[0, 0, :] = 0.0
    if W > 2:
        load[0, 1, :] = 1e4                 # beyond every capacity: no feasible candidate
    return wl, prof, sp, load


def _check_totals(sp, prof, out, ref, fixed_idx, J):
    nj, tj = oracle.config_tables(sp.n_max, prof.tp, sp.F)
    tot = oracle.totals(ref["best_idx"], ref["best_E"], J, nj, tj)
    assert np.array_equal(out["n_infeasible"].astype(np.int64), tot["n_infeasible"].astype(np.int64))
    assert np.allclose(out["E_total"], tot["E_total"], rtol=REL_TOL, atol=0)
    if out["E_window"] is not None:
        assert np.allclose(out["E_window"], tot["E_window"], rtol=REL_TOL, atol=1e-12)
        assert np.allclose(out["E_window"].sum(axis=1), out["E_total"], rtol=1e-12)
    # histogram and GPU counts recomputed from the GPU's own indices must match what it reported;
    # with the oracle's choice substituted on exempted tiles they must match the oracle
    if out["hist"] is not None:
        S = fixed_idx.shape[0]
        own = np.stack([np.bincount(out["best_idx"][s][out["best_idx"][s] >= 0], minlength=J) for s in range(S)])
        assert np.array_equal(out["hist"].astype(np.int64), own)
        sub = np.stack([np.bincount(fixed_idx[s][fixed_idx[s] >= 0], minlength=J) for s in range(S)])
        assert np.array_equal(sub, tot["hist"].astype(np.int64))
    if out["gpus"] is not None:
        idx = out["best_idx"]
        g = np.where(idx >= 0, nj[np.maximum(idx, 0)] * tj[np.maximum(idx, 0)], 0).sum(axis=2)
        assert np.array_equal(out["gpus"].astype(np.int64), g)


CASES = [
    dict(name="cfg1", W=61, S=2),                              # J = 336, 16 instance counts: half-warp groups
    dict(name="cfg2", W=45, S=2),                              # J = 2048, two instance counts per lane
    dict(name="cfg3", W=70, S=1),                              # J = 1024, one instance count per lane
    dict(name="cfg5", W=3, S=1),                               # J = 80896, off-grid f, M = 64: tables read through L1
    dict(name="cfg2", W=33, S=1, n_max=100, seed=3),           # ragged: 100 instance counts -> 4 per lane, some idle
    dict(name="cfg2", W=20, S=1, n_max=5, seed=4),             # 8-lane groups
    dict(name="cfg1", W=20, S=1, n_max=1, seed=5),             # a single instance count
    dict(name="cfg2", W=25, S=2, budget=24, seed=6),           # Eq. 1 GPU budget
    dict(name="cfg1", W=25, S=1, paper_slo=True, seed=7),      # per-class SLOs of the thresholds table
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
def test_eval_select_small(dyn, case):
    wl, prof, sp, load = _small(**case)
    J = sp.n_max * prof.T * sp.F
    ref = oracle.eval_select(prof, sp, load)
    out = out_to_host(gpu_eval_select(dyn, prof, sp, load))
    fixed, n_ex = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref)
    _check_totals(sp, prof, out, ref, fixed, J)
    assert (ref["best_idx"] >= 0).sum() > 0.3 * ref["best_idx"].size


ODD = [dict(name="cfg2", W=9, S=1, n_max=7, budget=20, seed=8),       # odd instance count under a GPU budget
       dict(name="cfg3", W=9, S=1, n_max=33, seed=9)]                 # odd, more than a warp of counts


@pytest.mark.parametrize("case", CASES + ODD, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
def test_eval_configs_then_select_small(dyn, case):
    wl, prof, sp, load = _small(**case)
    if case["name"] == "cfg5":
        load = load[:, :2]
    S, W, Cn = load.shape
    J = sp.n_max * prof.T * sp.F
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load).cuda()
    d_E = torch.full((S, W, Cn, J), -7.0, dtype=torch.float32, device="cuda")
    ws = torch.empty(dyn.dyn_workspace_bytes(p, s, S, W), dtype=torch.uint8, device="cuda")
    dyn.dyn_eval_configs(p, s, d_load, d_E, ws)
    torch.cuda.synchronize()
    E = d_E.cpu().numpy()
    ref = oracle.eval_configs(prof, sp, load)
    fin_r, fin_g = np.isfinite(ref), np.isfinite(E)
    both = fin_r & fin_g
    rel = np.abs(E[both] - ref[both]) / np.abs(ref[both])
    assert rel.max() <= REL_TOL
    assert (E[~fin_g] == np.inf).all()
    # feasibility may differ only where a deciding quantity sits within REL_TOL of its bound
    diff = np.argwhere(fin_r != fin_g)
    assert len(diff) <= 1e-4 * E.size + 2
    for s_, w_, c_, j_ in diff:
        _, tb, _, u, _ = oracle.eval_tile(prof, sp, int(c_), float(load[s_, w_, c_]), details=True)
        slo = float(sp.slo_tbt_s[c_])
        assert min(abs(tb[j_] - slo) / slo, abs(u[j_] - 1.0)) < REL_TOL

    # stage (c) on the GPU's own tensor: bit-exact against the oracle's argmin of the same numbers
    out = dyn.SelectOut(S, W, Cn, J)
    ws2 = torch.empty(dyn.dyn_select_workspace_bytes(S, W, J), dtype=torch.uint8, device="cuda")
    nj, tj = oracle.config_tables(sp.n_max, prof.tp, sp.F)
    dyn.dyn_select(d_E, out, ws2, nj, tj)
    torch.cuda.synchronize()
    o = out_to_host(out)
    idx, be, _ = oracle.select(E.astype(np.float64))
    assert np.array_equal(o["best_idx"], idx)
    assert np.array_equal(o["best_E"].astype(np.float64), be)
    tot = oracle.totals(idx, be, J, nj, tj)
    assert np.array_equal(o["n_infeasible"].astype(np.int64), tot["n_infeasible"].astype(np.int64))
    assert np.allclose(o["E_total"], tot["E_total"], rtol=1e-12)
    assert np.allclose(o["E_window"], tot["E_window"], rtol=1e-12, atol=0)
    assert np.array_equal(o["hist"].astype(np.int64), tot["hist"].astype(np.int64))
    assert np.array_equal(o["gpus"].astype(np.int64), tot["gpus"].astype(np.int64))


@pytest.mark.parametrize("large", [False, True], ids=["tables-in-shared-memory", "tables-per-class"])
@pytest.mark.parametrize("monotone", [False, True], ids=["tbt-rises-and-falls", "tbt-never-decreases"])
def test_eval_select_free_form_tables(dyn, monotone, large):
    """Both evaluation paths of the fused kernel: per-candidate TBT interpolation when some table row
    decreases with load, the load-threshold path when none does; with all classes' tables staged at
    once, and with the per-class kernel that larger tables need."""
    prof, sp = random_tables(17, monotone, large)
    load = gen.random_loads((2, 37 if not large else 11, 9), seed=5, mean=6.0)
    J = sp.n_max * prof.T * sp.F
    ref = oracle.eval_select(prof, sp, load)
    out = out_to_host(gpu_eval_select(dyn, prof, sp, load))
    fixed, n_ex = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref)
    _check_totals(sp, prof, out, ref, fixed, J)
    feas = (ref["best_idx"] >= 0).mean()
    assert 0.2 < feas <= 1.0


@pytest.mark.parametrize("budget", [0, 60], ids=["no-budget", "gpu-budget"])
@pytest.mark.parametrize("large", [False, True], ids=["tables-in-shared-memory", "tables-per-class"])
def test_few_rows_without_a_load_threshold(dyn, large, budget):
    """The evaluation path is chosen per table row: a profile whose TBT rows rise with load except for a few that
    cross the SLO twice keeps the load-threshold path for all other rows (dips that stay on one side of the SLO
    included) and interpolates TBT per candidate only for those few.  Fused kernel and evaluate-only kernel."""
    prof, sp, bad = tables_with_few_rows_without_threshold(23, large)
    assert len(bad) >= 3
    sp = gen.make_space(sp.f_cand_mhz, sp.n_max, sp.window_s, slo_ttft=0.8, slo_tbt=0.1, gpu_budget=budget)
    load = gen.random_loads((2, 29 if not large else 7, 9), seed=6, mean=6.0)
    J = sp.n_max * prof.T * sp.F
    ref = oracle.eval_select(prof, sp, load)
    out = out_to_host(gpu_eval_select(dyn, prof, sp, load))
    fixed, n_ex = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref)
    _check_totals(sp, prof, out, ref, fixed, J)
    # the rows that need the general path do get chosen somewhere (otherwise the case tests nothing)
    jbest = ref["best_idx"]
    tq = (jbest % (prof.T * sp.F))[jbest >= 0]
    cls = np.broadcast_to(np.arange(9), jbest.shape)[jbest >= 0]
    chosen_t = set(zip(cls.tolist(), (tq // sp.F).tolist()))
    assert any((c, t) in chosen_t for c, t, _ in bad)
    # evaluate-only kernel on the same tables
    S, W, Cn = load.shape
    W2 = min(W, 3)
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load[:, :W2].copy()).cuda()
    d_E = torch.empty((S, W2, Cn, J), dtype=torch.float32, device="cuda")
    ws = torch.empty(dyn.dyn_workspace_bytes(p, s, S, W2), dtype=torch.uint8, device="cuda")
    dyn.dyn_eval_configs(p, s, d_load, d_E, ws)
    torch.cuda.synchronize()
    E = d_E.cpu().numpy()
    refE = oracle.eval_configs(prof, sp, load[:, :W2])
    fin_r, fin_g = np.isfinite(refE), np.isfinite(E)
    both = fin_r & fin_g
    assert (np.abs(E[both] - refE[both]) / np.abs(refE[both])).max() <= REL_TOL
    diff = np.argwhere(fin_r != fin_g)
    assert len(diff) <= 1e-4 * E.size + 2
    for s_, w_, c_, j_ in diff:
        _, tb, _, u, _ = oracle.eval_tile(prof, sp, int(c_), float(load[s_, w_, c_]), details=True)
        assert min(abs(tb[j_] - 0.1) / 0.1, abs(u[j_] - 1.0)) < REL_TOL


def test_self_check_passes_on_this_build(dyn):
    dyn.dyn_self_check()                      # raises when subnormal arithmetic is flushed to zero


def test_limits_of_the_candidate_space(dyn):
    """Largest built shape per axis (256 instance counts, 16 TP degrees) and the smallest tables
    (two frequency rows, two load knots); the GPU budget cuts the space unevenly."""
    rng = np.random.default_rng(3)
    Cn, T, R, M = 9, 16, 2, 2
    tp = np.arange(1, T + 1, dtype=np.int32)
    fg = np.array([800.0, 1980.0], np.float32)
    ttft = (0.1 + 0.5 * rng.random((Cn, T, R))).astype(np.float32)
    cap = (0.5 + 2.0 * rng.random((Cn, T, R))).astype(np.float32)
    tbt = np.sort(0.05 + 0.08 * rng.random((Cn, T, R, M)), axis=-1).astype(np.float32)
    pw = (100 + 50 * tp[None, :, None, None] * (1 + rng.random((Cn, T, R, M)))).astype(np.float32)
    prof = gen.Profile(tp, fg, ttft, cap, tbt, pw)
    cand = np.linspace(800, 1980, 16).astype(np.float32)
    for budget in (0, 300):
        sp = gen.make_space(cand, 256, 5.0, slo_ttft=0.5, slo_tbt=0.1, gpu_budget=budget)
        load = gen.random_loads((1, 7, 9), seed=2, mean=40.0)
        J = 256 * T * 16
        ref = oracle.eval_select(prof, sp, load)
        out = out_to_host(gpu_eval_select(dyn, prof, sp, load))
        fixed, _ = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref)
        _check_totals(sp, prof, out, ref, fixed, J)
        assert (ref["best_idx"] >= 0).all()


def test_loads_that_are_not_valid_numbers_count_as_zero(dyn):
    wl, prof, sp, load = _small("cfg1", W=6, seed=12)
    bad = load.copy()
    bad[0, 2, 0] = -3.0
    bad[0, 2, 1] = np.nan
    bad[0, 3, 4] = -np.inf
    clean = bad.copy()
    clean[0, 2, 0] = clean[0, 2, 1] = clean[0, 3, 4] = 0.0
    a = out_to_host(gpu_eval_select(dyn, prof, sp, bad))
    b = out_to_host(gpu_eval_select(dyn, prof, sp, clean))
    assert np.array_equal(a["best_idx"], b["best_idx"]) and np.array_equal(a["best_E"], b["best_E"])
    ref = oracle.eval_select(prof, sp, clean)
    check_selection(prof, sp, clean, a["best_idx"], a["best_E"], ref)


def test_kernel_timing_events(dyn):
    """The instrumentation hook brackets the sweep kernel: a positive time, shorter than the whole call."""
    wl, prof, sp, load = _small("cfg2", W=300, S=2, seed=13)
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load).cuda()
    out = dyn.SelectOut(2, 300, 9, wl.J)
    ws = torch.empty(dyn.dyn_workspace_bytes(p, s, 2, 300), dtype=torch.uint8, device="cuda")
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0.record(); k1.record()
    dyn.dyn_eval_select(p, s, d_load, out, ws)                 # warm-up
    torch.cuda.synchronize()
    dyn.dyn_set_timing_events(k0, k1)
    c0.record()
    dyn.dyn_eval_select(p, s, d_load, out, ws)
    c1.record()
    dyn.dyn_set_timing_events(None, None)
    torch.cuda.synchronize()
    assert 0.0 < k0.elapsed_time(k1) <= c0.elapsed_time(c1)
    # switched off again: a later call leaves the events alone
    before = k0.elapsed_time(k1)
    dyn.dyn_eval_select(p, s, d_load, out, ws)
    torch.cuda.synchronize()
    assert k0.elapsed_time(k1) == before


def test_select_ties_infeasible_and_odd_sizes(dyn):
    """dyn_select alone: exact duplicates -> lowest index; all +inf -> -1; J not a multiple of 4."""
    rng = np.random.default_rng(0)
    for J in (1, 3, 37, 336, 1001):
        S, W, Cn = 2, 9, 5
        E = (np.round(rng.random((S, W, Cn, J)) * 16) / 8).astype(np.float32)
        E[rng.random(E.shape) < 0.5] = np.inf
        E[0, 0] = np.inf
        E[1, 2, 3] = 2.5
        d_E = torch.from_numpy(E).cuda()
        out = dyn.SelectOut(S, W, Cn, J, gpus=False)
        ws = torch.empty(dyn.dyn_select_workspace_bytes(S, W, J), dtype=torch.uint8, device="cuda")
        dyn.dyn_select(d_E, out, ws)
        torch.cuda.synchronize()
        o = out_to_host(out)
        idx, be, _ = oracle.select(E.astype(np.float64))
        assert np.array_equal(o["best_idx"], idx)
        assert np.array_equal(o["best_E"].astype(np.float64), be)
        assert o["best_idx"][1, 2, 3] == 0 and (o["best_idx"][0, 0] == -1).all()
        tot = oracle.totals(idx, be, J)
        assert np.array_equal(o["hist"].astype(np.int64), tot["hist"].astype(np.int64))
        assert np.allclose(o["E_total"], tot["E_total"], rtol=1e-12)


def test_paper_tables_through_the_gpu_select(dyn, golden_dir):
    """Tables 1-3 of the paper as energy rows: the kernel picks the bold cell of every row."""
    import os
    rows = []
    for line in open(os.path.join(golden_dir, "paper_energy_tables.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            _, _, cells, col = [x.strip() for x in line.split(";")]
            rows.append(([np.inf if v == "x" else float(v) for v in cells.split()], int(col)))
    E = np.array([r[0] for r in rows], dtype=np.float32).reshape(1, 2, 9, 12)
    out = dyn.SelectOut(1, 2, 9, 12, gpus=False)
    ws = torch.empty(dyn.dyn_select_workspace_bytes(1, 2, 12), dtype=torch.uint8, device="cuda")
    dyn.dyn_select(torch.from_numpy(E).cuda(), out, ws)
    torch.cuda.synchronize()
    assert out.best_idx.cpu().numpy().ravel().tolist() == [r[1] for r in rows]


def test_determinism_and_empty_shapes(dyn):
    wl, prof, sp, load = _small("cfg2", W=2100, S=1, n_max=8, seed=11)       # two partial-sum chunks
    a = out_to_host(gpu_eval_select(dyn, prof, sp, load))
    b = out_to_host(gpu_eval_select(dyn, prof, sp, load))
    assert a["E_total"].tobytes() == b["E_total"].tobytes()
    assert a["E_window"].tobytes() == b["E_window"].tobytes()
    assert np.array_equal(a["best_idx"], b["best_idx"])
    ref = oracle.eval_select(prof, sp, load)
    fixed, _ = check_selection(prof, sp, load, a["best_idx"], a["best_E"], ref)
    _check_totals(sp, prof, a, ref, fixed, sp.n_max * prof.T * sp.F)
    # zero scenarios / zero windows: nothing to do, no error
    p, s = gpu_profile_space(dyn, prof, sp)
    ws = torch.empty(max(256, dyn.dyn_workspace_bytes(p, s, 0, 0)), dtype=torch.uint8, device="cuda")
    out = dyn.SelectOut(0, 0, 9, 8 * 32)
    dyn.dyn_eval_select(p, s, torch.empty((0, 0, 9), dtype=torch.float32, device="cuda"), out, ws)
    torch.cuda.synchronize()


def test_argument_errors(dyn):
    wl, prof, sp, load = _small("cfg1", W=4)
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load).cuda()
    out = dyn.SelectOut(1, 4, 9, wl.J)
    nb = dyn.dyn_workspace_bytes(p, s, 1, 4)
    assert nb > 0 and nb % 256 == 0
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select(p, s, d_load, out, torch.empty(nb - 256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == dyn.DYN_EWORKSPACE
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select(p, s, d_load, out, None)
    assert e.value.status == dyn.DYN_EWORKSPACE
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    bad = dyn.Space(np.array([700.0, 900.0], np.float32), 4, sp.slo_ttft_s, sp.slo_tbt_s, 60.0)
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select(p, bad, d_load, dyn.SelectOut(1, 4, 9, 4 * 3 * 2), ws)
    assert e.value.status == dyn.DYN_EUNSUPPORTED
    bad = dyn.Space(np.array([1200.0, 900.0], np.float32), 4, sp.slo_ttft_s, sp.slo_tbt_s, 60.0)
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select(p, bad, d_load, dyn.SelectOut(1, 4, 9, 4 * 3 * 2), ws)
    assert e.value.status == dyn.DYN_EINVAL
    bad = dyn.Space(sp.f_cand_mhz, 0, sp.slo_ttft_s, sp.slo_tbt_s, 60.0)
    with pytest.raises(dyn.DynError):
        dyn.dyn_eval_select(p, bad, d_load, out, ws)
    # the library is still usable after the rejected calls
    dyn.dyn_eval_select(p, s, d_load, out, ws)
    torch.cuda.synchronize()
    assert int((out.best_idx >= -1).sum().item()) == 36
