"""GPU parity at the benchmark's full sizes, in the launch configuration the benchmark times."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import REL_TOL, check_selection, gpu_bin_trace, gpu_eval_select, out_to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _pipeline(dyn, name):
    wl = gen.workload(name)
    t, i, o = gen.make_trace(wl.trace)
    W = wl.trace.n_windows
    counts, load, dropped = gpu_bin_trace(dyn, t, i, o, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    ref_c, ref_d = oracle.bin_trace(t, i, o, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    assert np.array_equal(counts, ref_c) and dropped == ref_d
    ref_load = oracle.load_from_counts(ref_c, wl.window_s)
    assert np.array_equal(load, ref_load)
    return wl, ref_c, ref_load


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg3code", "cfg5"])
def test_full_pipeline(dyn, name):
    """trace -> counts -> loads -> fused evaluate+select -> totals, every tile checked."""
    wl, counts, load = _pipeline(dyn, name)
    prof, sp = wl.profile(), wl.space()
    load = load[None]
    ref = oracle.eval_select(prof, sp, load)
    out = out_to_host(gpu_eval_select(dyn, prof, sp, load, hist=True, gpus=True))
    fixed, n_ex = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref, max_exempt_frac=2e-3)
    nj, tj = oracle.config_tables(sp.n_max, prof.tp, sp.F)
    tot = oracle.totals(ref["best_idx"], ref["best_E"], wl.J, nj, tj)
    assert np.allclose(out["E_total"], tot["E_total"], rtol=REL_TOL)
    assert np.array_equal(out["n_infeasible"].astype(np.int64), tot["n_infeasible"].astype(np.int64))
    assert int(out["hist"].sum()) == load.size - int(out["n_infeasible"].sum())


def test_monte_carlo_scenarios_sampled(dyn):
    """4096 Poisson-resampled day-long scenarios on the GPU; the oracle recomputes 66 of them, spread evenly over
    the batch, tile by tile, and per-scenario invariants are checked on all."""
    wl, counts, load0 = _pipeline(dyn, "cfg2")
    prof, sp = wl.profile(), wl.space()
    S = 4096
    cs = gen.resample_counts(counts, S, seed=4)
    assert np.array_equal(cs[0], counts)
    load = oracle.load_from_counts(cs, wl.window_s)
    out = gpu_eval_select(dyn, prof, sp, load, windows=False, hist=True, gpus=False)
    o = out_to_host(out)
    W, Cn = counts.shape
    assert (o["hist"].sum(axis=1) == W * Cn - o["n_infeasible"]).all()
    fin = np.where(o["best_idx"] >= 0, o["best_E"].astype(np.float64), 0.0).sum(axis=(1, 2))
    assert np.allclose(o["E_total"], fin, rtol=1e-9)
    sample = sorted(set(np.linspace(0, S - 1, 64).astype(int).tolist()) | {1, 77})       # 64 strata and two more
    assert len(sample) >= 64
    ref = oracle.eval_select(prof, sp, load[sample])
    fixed, n_ex = check_selection(prof, sp, load[sample], o["best_idx"][sample], o["best_E"][sample], ref,
                                  max_exempt_frac=2e-3)
    tot = oracle.totals(ref["best_idx"], ref["best_E"], wl.J)
    assert np.allclose(o["E_total"][sample], tot["E_total"], rtol=REL_TOL)
    for k, s in enumerate(sample):
        sub = np.bincount(fixed[k][fixed[k] >= 0], minlength=wl.J)
        assert np.array_equal(sub, tot["hist"][k].astype(np.int64))


@pytest.mark.parametrize("which", ["one", "all"], ids=["one-row-without-threshold", "every-feasible-row-without-threshold"])
def test_day_shape_with_rows_that_cross_the_slo_twice(dyn, which):
    """The 1-day shape at full size (1440 windows x 9 classes x 2048 candidates, 8 scenarios) on a profile whose TBT
    rows leave the SLO and return to it as the load grows: one such row (the other rows keep their load threshold,
    the kernel serves that row in its second loop) or every row that is feasible at all (the kernel interpolates TBT
    for every candidate).  Every tile against the oracle."""
    wl, counts, load0 = _pipeline(dyn, "cfg2")
    prof, sp = wl.profile(), wl.space()
    tbt = prof.tbt.copy()
    n = 0
    for c in range(9):
        slo = float(sp.slo_tbt_s[c])
        for t, r in np.argwhere((tbt[c, :, :, 0] <= slo) & (tbt[c, :, :, 2] <= slo)):
            if which == "one" and n >= 1:
                break
            tbt[c, t, r, 1] = 1.05 * slo                      # feasible, infeasible, feasible again
            n += 1
    assert n == 1 if which == "one" else n > 100
    prof = gen.Profile(prof.tp, prof.f_grid_mhz, prof.ttft, prof.cap, tbt, prof.pow)
    cs = gen.resample_counts(counts, 8, seed=4)
    load = oracle.load_from_counts(cs, wl.window_s)
    ref = oracle.eval_select(prof, sp, load)
    out = out_to_host(gpu_eval_select(dyn, prof, sp, load, hist=True, gpus=False))
    fixed, n_ex = check_selection(prof, sp, load, out["best_idx"], out["best_E"], ref, max_exempt_frac=2e-3)
    tot = oracle.totals(ref["best_idx"], ref["best_E"], wl.J)
    assert np.allclose(out["E_total"], tot["E_total"], rtol=REL_TOL)
    assert np.array_equal(out["n_infeasible"].astype(np.int64), tot["n_infeasible"].astype(np.int64))
    # the changed rows matter: some tile's choice differs from the unchanged profile's
    base = oracle.eval_select(wl.profile(), sp, load[:1])
    if which == "all":
        assert (base["best_idx"] != ref["best_idx"][:1]).any()
