"""GPU parity of the selection with re-configuration costs against the oracle.  Several schedules can be within
rounding of the optimum, so what is compared is what is unique: the minimised total (1e-5), which (scenario,
class) pairs have a schedule, and that the GPU's own schedule is valid: its states reproduce its reported window
energies and its reported total, and that total is optimal within the tolerance."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import REL_TOL, gpu_profile_space

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _run(dyn, prof, sp, R, load):
    S, W, Cn = load.shape
    p, s = gpu_profile_space(dyn, prof, sp)
    J = sp.n_max * prof.T * sp.F
    out = dyn.SelectOut(S, W, Cn, J, windows=False, hist=False, gpus=False)
    total = torch.full((S, Cn), -7.0, dtype=torch.float64, device="cuda")
    ws = torch.empty(dyn.dyn_reconf_workspace_bytes(p, s, S, W), dtype=torch.uint8, device="cuda")
    dyn.dyn_reconf_select(p, s, torch.from_numpy(R).cuda(), torch.from_numpy(load).cuda(), out, total, ws)
    torch.cuda.synchronize()
    return out, total.cpu().numpy()


def _check(dyn, prof, sp, R, load):
    S, W, Cn = load.shape
    F, T = sp.F, prof.T
    ref = oracle.reconf_select(prof, sp, R, load)
    out, total = _run(dyn, prof, sp, R, load)
    idx, E = out.best_idx.cpu().numpy(), out.best_E.cpu().numpy()
    have = np.isfinite(ref["path_total"])
    assert (np.isfinite(total) == have).all()
    assert ((idx >= 0).all(axis=1) == have).all() and ((idx < 0).all(axis=1) == ~have).all()
    assert np.isinf(E[idx < 0]).all()
    np.testing.assert_allclose(total[have], ref["path_total"][have], rtol=REL_TOL)
    same = 0
    for s, c in zip(*np.nonzero(have)):
        st = idx[s, :, c] // F
        # window energies of the GPU's states, from the oracle's per-candidate values
        want = np.array([oracle.eval_tile(prof, sp, int(c), float(load[s, w, c]))[idx[s, w, c]] for w in range(W)])
        np.testing.assert_allclose(E[s, :, c], want, rtol=REL_TOL)
        again = want.sum() + sum(float(R[a, b]) for a, b in zip(st, st[1:]))
        assert again <= ref["path_total"][s, c] * (1 + REL_TOL)            # the schedule is optimal within tolerance
        assert total[s, c] == pytest.approx(again, rel=REL_TOL)            # and the reported total is its cost
        same += int((idx[s, :, c] == ref["best_idx"][s, :, c]).all())
    fin = np.where(idx >= 0, E.astype(np.float64), 0.0).sum(axis=(1, 2))
    np.testing.assert_allclose(out.E_total.cpu().numpy(), fin, rtol=1e-12)
    assert (out.n_infeasible.cpu().numpy() == (idx < 0).sum(axis=(1, 2))).all()
    return same, int(have.sum())


def _table(NS, seed, scale):
    R = np.random.default_rng(seed).uniform(0.0, scale, (NS, NS)).astype(np.float32)
    np.fill_diagonal(R, 0.0)
    return R


def test_hour_trace_shape(dyn):
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), gen.make_space(wl.f_cand_mhz, 16, wl.window_s)
    NS = sp.n_max * prof.T
    load = gen.random_loads((2, 60, 9), seed=51, mean=2.0, zero_frac=0.0)
    same, n = _check(dyn, prof, sp, _table(NS, 1, 3.0), load)
    assert n >= 9 and same >= n // 2                        # most schedules are reproduced state for state


def test_many_states_with_budget_and_ragged_sizes(dyn):
    """NS = 37 * 4 states (not a multiple of 32), 45 windows (not a multiple of the eight windows the walk back
    looks ahead), a GPU budget that rules out part of the states."""
    wl = gen.workload("cfg2")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, 37, wl.window_s, gpu_budget=48)
    load = gen.random_loads((2, 45, 9), seed=52, mean=3.0, zero_frac=0.0)
    _check(dyn, prof, sp, _table(sp.n_max * prof.T, 2, 10.0), load)


def test_free_and_prohibitive_tables(dyn):
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), gen.make_space(wl.f_cand_mhz, 8, wl.window_s)
    NS = sp.n_max * prof.T
    load = gen.random_loads((1, 33, 9), seed=53, mean=1.5, zero_frac=0.0)
    load[0, 5, 8] = 1e6                                     # no state carries this: class 8 has no schedule
    _check(dyn, prof, sp, np.zeros((NS, NS), np.float32), load)
    wall = np.full((NS, NS), 1e9, np.float32)
    np.fill_diagonal(wall, 0.0)
    _check(dyn, prof, sp, wall, load)
    out, total = _run(dyn, prof, sp, wall, load)
    st = out.best_idx.cpu().numpy()[0] // sp.F
    assert np.isinf(total[0, 8]) and (st[:, 8] < 0).all()
    assert all(len(set(st[:, c].tolist())) == 1 for c in range(8))          # one sharding for the whole horizon


def test_single_window_and_errors(dyn):
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), gen.make_space(wl.f_cand_mhz, 4, wl.window_s)
    NS = sp.n_max * prof.T
    _check(dyn, prof, sp, _table(NS, 3, 1.0), gen.random_loads((1, 1, 9), seed=54, mean=1.0, zero_frac=0.0))
    p, s = gpu_profile_space(dyn, prof, gen.make_space(wl.f_cand_mhz, 400, wl.window_s))
    out = dyn.SelectOut(1, 1, 9, 1, windows=False, hist=False, gpus=False)
    tot = torch.zeros((1, 9), dtype=torch.float64, device="cuda")
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(dyn.DynError) as e:                  # Nmax beyond the built limit
        dyn.dyn_reconf_select(p, s, torch.zeros((4, 4), device="cuda"), torch.zeros((1, 1, 9), device="cuda"), out, tot, ws)
    assert e.value.status == dyn.DYN_EUNSUPPORTED
    p, s = gpu_profile_space(dyn, prof, sp)
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_reconf_select(p, s, torch.zeros((NS, NS), device="cuda"), torch.zeros((1, 1, 9), device="cuda"), out, tot,
                              ws[:256])
    assert e.value.status == dyn.DYN_EWORKSPACE


@pytest.mark.parametrize("n_max,W", [(5, 19), (7, 9)])
def test_state_counts_that_are_not_multiples_of_four(dyn, n_max, W):
    """TP 2/4/8 with 5 or 7 instance counts: 15 and 21 states (padded vector entries, ragged rows of the table)."""
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), gen.make_space(wl.f_cand_mhz, n_max, wl.window_s)
    load = gen.random_loads((2, W, 9), seed=55 + n_max, mean=0.8, zero_frac=0.0)
    _check(dyn, prof, sp, _table(n_max * prof.T, 4, 2.0), load)


def test_more_states_than_fit_on_chip(dyn):
    """400 states: the overhead table (640 KB) only partly fits in shared memory and registers, the rest is read
    from global memory; the walk back takes its plain path (more than 256 states)."""
    wl = gen.workload("cfg2")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, 100, wl.window_s)
    load = gen.random_loads((1, 12, 9), seed=56, mean=6.0, zero_frac=0.0)
    _check(dyn, prof, sp, _table(400, 5, 8.0), load)


@pytest.mark.parametrize("monotone", [False, True], ids=["tbt-rises-and-falls", "tbt-never-decreases"])
def test_free_form_tables(dyn, monotone):
    """Profiles that are not the closed forms (per-pair TTFT misses, TBT that rises and falls with load)."""
    from parity import random_tables
    prof, sp0 = random_tables(31, monotone)
    sp = gen.make_space(sp0.f_cand_mhz, 12, 60.0, slo_ttft=0.8, slo_tbt=0.1)
    load = gen.random_loads((1, 14, 9), seed=57, mean=6.0, zero_frac=0.0)
    _check(dyn, prof, sp, _table(sp.n_max * prof.T, 6, 4.0), load)


@pytest.mark.parametrize("kind", ["cheap-next-to-the-cost-spread", "few-cheap-moves", "staying-costs-too"])
def test_tables_that_let_the_forward_pass_skip_sources(dyn, kind):
    """The forward pass skips sources that cannot attain any minimum (a bound from the state of the last minimum and
    the row extremes of the table).  Tables with small entries (nearly every source is skipped), with a few cheap
    moves among prohibitive ones (the row minima are far below the row maxima) and with a non-zero diagonal must give
    the optimum of the full scan, which the oracle does."""
    wl = gen.workload("cfg2")
    prof, sp = wl.profile(), gen.make_space(wl.f_cand_mhz, 24, wl.window_s)
    NS = sp.n_max * prof.T
    rng = np.random.default_rng(61)
    if kind == "cheap-next-to-the-cost-spread":
        R = rng.uniform(0.0, 0.5, (NS, NS)).astype(np.float32)
        np.fill_diagonal(R, 0.0)
    elif kind == "few-cheap-moves":
        R = np.full((NS, NS), 5e3, np.float32)
        cheap = rng.random((NS, NS)) < 0.05
        R[cheap] = rng.uniform(0.0, 3.0, int(cheap.sum())).astype(np.float32)
        np.fill_diagonal(R, 0.0)
    else:
        R = rng.uniform(1.0, 4.0, (NS, NS)).astype(np.float32)              # the diagonal too: no move is free
    load = gen.random_loads((2, 40, 9), seed=62, mean=3.0)
    _check(dyn, prof, sp, R, load)
