"""GPU parity of the mixed-parallelism pools (Eq. 1 in full) against the oracle: chosen counts, frequencies
and tuple number identical except where the oracle's best and runner-up tuples are within 1e-5 or a deciding
quantity of the tile is within 1e-5 of its bound; energies within 1e-5; totals of the GPU's own choice."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import REL_TOL, gpu_eval_select, gpu_profile_space

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _run(dyn, prof, sp, load):
    S, W, Cn = load.shape
    p, s = gpu_profile_space(dyn, prof, sp)
    out = dyn.MixedOut(S, W, Cn, prof.T)
    for t in (out.counts, out.freq, out.tuple):
        t.fill_(-7)
    ws = torch.empty(dyn.dyn_mixed_workspace_bytes(p, s, S, W), dtype=torch.uint8, device="cuda")
    dyn.dyn_mixed_select(p, s, torch.from_numpy(load).cuda(), out, ws)
    torch.cuda.synchronize()
    return out


def _check(dyn, prof, sp, load, max_exempt=0.01):
    ref = oracle.mixed_select(prof, sp, load)
    out = _run(dyn, prof, sp, load)
    cnt, frq, tup = out.counts.cpu().numpy(), out.freq.cpu().numpy(), out.tuple.cpu().numpy()
    E = out.best_E.cpu().numpy()
    with np.errstate(invalid="ignore"):                     # inf - inf on tiles without a feasible tuple
        gap = np.where(ref["tuple_no"] >= 0, (ref["E2"] - ref["best_E"]) / np.maximum(ref["best_E"], 1e-300), np.inf)
    exempt = (gap < REL_TOL) | (ref["margin"] < REL_TOL)
    same = (tup == ref["tuple_no"]) & (cnt == ref["counts"]).all(axis=3) & (frq == ref["freq"]).all(axis=3)
    assert (same | exempt).all(), f"{(~(same | exempt)).sum()} tiles differ without a near-tie or near-bound"
    assert (~same).sum() <= max(3, max_exempt * same.size)
    ok = same & (ref["tuple_no"] >= 0)
    if ok.any():
        rel = np.abs(E[ok].astype(np.float64) - ref["best_E"][ok]) / ref["best_E"][ok]
        assert rel.max() <= REL_TOL, f"energy off by {rel.max():.3e}"
    none = same & (ref["tuple_no"] < 0)
    assert np.isinf(E[none]).all() and (cnt[none] == -1).all() and (frq[none] == -1).all()
    # the GPU's own choice is consistent: within budget, frequencies exactly where counts are positive
    feas = tup >= 0
    gp = (cnt * prof.tp[None, None, None, :]).sum(axis=3)
    assert (gp[feas] <= sp.gpu_budget).all() and (gp[feas] > 0).all()
    assert ((cnt > 0) == (frq >= 0))[feas].all()
    fin = np.where(feas, E.astype(np.float64), 0.0).sum(axis=(1, 2))
    np.testing.assert_allclose(out.E_total.cpu().numpy(), fin, rtol=1e-12)
    assert (out.n_infeasible.cpu().numpy() == (~feas).sum(axis=(1, 2))).all()
    return ref, out


def test_hour_trace_shape_three_parallelisms(dyn):
    """cfg1's profile (TP 2/4/8, 7 frequencies), 32 GPUs per pool, up to 16 instances per parallelism."""
    wl = gen.workload("cfg1")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, 16, wl.window_s, gpu_budget=32)
    load = gen.random_loads((3, 60, 9), seed=31, mean=3.0)
    load[0, 0, :] = 0.0
    load[1, 1, :] = 500.0                                   # nothing carries this
    ref, out = _check(dyn, prof, sp, load)
    assert (ref["tuple_no"][1, 1] == -1).all()
    assert ((ref["counts"] > 0).sum(axis=3) > 1).any()      # some pools do mix parallelisms


def test_four_parallelisms_jittered_profile_small_budget(dyn):
    wl = gen.workload("cfg2")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, 6, wl.window_s, gpu_budget=12)
    load = gen.random_loads((2, 40, 9), seed=32, mean=1.5)
    _check(dyn, prof, sp, load)


def test_paper_slos_and_off_grid_frequencies(dyn):
    """Per-class TTFT SLOs of the thresholds table; candidates between the profiled frequencies."""
    wl = gen.workload("cfg1")
    prof = wl.profile()
    st, sb = gen.paper_slos()
    fc = np.array([850, 1111, 1500, 1900], np.float32)
    sp = gen.make_space(fc, 8, 30.0, slo_ttft=st, slo_tbt=sb, gpu_budget=24)
    load = gen.random_loads((2, 30, 9), seed=33, mean=2.0)
    _check(dyn, prof, sp, load)


def test_single_parallelism_equals_single_type_selection(dyn):
    """One TP degree: the tuple is the instance count, so the fused single-type call gives the same choice."""
    wl = gen.workload("cfg1")
    prof1 = gen.make_profile((4,), wl.f_grid_mhz, wl.M, gen.class_coefficients(3))
    sp = gen.make_space(wl.f_cand_mhz, 12, 60.0, gpu_budget=40)
    load = gen.random_loads((2, 20, 9), seed=34, mean=3.0)
    ref, out = _check(dyn, prof1, sp, load)
    single = gpu_eval_select(dyn, prof1, sp, load, windows=False, hist=False, gpus=False)
    idx = single.best_idx.cpu().numpy()
    cnt, frq = out.counts.cpu().numpy()[..., 0], out.freq.cpu().numpy()[..., 0]
    feas = idx >= 0
    agree = (cnt[feas] == idx[feas] // sp.F + 1) & (frq[feas] == idx[feas] % sp.F)
    assert agree.mean() > 0.99                              # the two kernels round differently at near-ties


def test_limits_and_errors(dyn):
    wl = gen.workload("cfg1")
    prof = wl.profile()
    p, s0 = gpu_profile_space(dyn, prof, gen.make_space(wl.f_cand_mhz, 4, 60.0))          # no budget
    assert dyn.dyn_mixed_workspace_bytes(p, s0, 1, 1) == 0 and dyn.dyn_mixed_tuple_count(p, s0) == 0
    out = dyn.MixedOut(1, 1, 9, 3)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_mixed_select(p, s0, torch.zeros((1, 1, 9), device="cuda"), out, ws)
    assert e.value.status == dyn.DYN_EINVAL
    # tuple count: TP 2/4/8, up to 4 each, 8 GPUs: brute force
    p, s1 = gpu_profile_space(dyn, prof, gen.make_space(wl.f_cand_mhz, 4, 60.0, gpu_budget=8))
    want = sum(1 for a in range(5) for b in range(5) for c in range(5) if 0 < 2 * a + 4 * b + 8 * c <= 8)
    assert dyn.dyn_mixed_tuple_count(p, s1) == want
    # too many tuples: 256^4 counts with a huge budget
    wl2 = gen.workload("cfg2")
    p2, s2 = gpu_profile_space(dyn, wl2.profile(), gen.make_space(wl2.f_cand_mhz, 255, 60.0, gpu_budget=10 ** 6))
    assert dyn.dyn_mixed_tuple_count(p2, s2) == 0
    out2 = dyn.MixedOut(1, 1, 9, 4)
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_mixed_select(p2, s2, torch.zeros((1, 1, 9), device="cuda"), out2, ws)
    assert e.value.status == dyn.DYN_EUNSUPPORTED
    # short workspace
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_mixed_select(p, s1, torch.zeros((1, 1, 9), device="cuda"), out, ws[:256])
    assert e.value.status == dyn.DYN_EWORKSPACE


@pytest.mark.parametrize("large", [False, True], ids=["tables-in-shared-memory", "tables-through-L1"])
@pytest.mark.parametrize("monotone", [False, True], ids=["tbt-rises-and-falls", "tbt-never-decreases"])
def test_free_form_tables(dyn, monotone, large):
    """Both variants of the kernel: the threshold variant needs every TBT row monotone and tables that fit in
    shared memory; a row that decreases somewhere, or larger tables, go to the plain variant."""
    from parity import random_tables
    prof, sp0 = random_tables(23, monotone, large)
    sp = gen.make_space(sp0.f_cand_mhz[::5] if large else sp0.f_cand_mhz, 6, 60.0, slo_ttft=0.8, slo_tbt=0.1, gpu_budget=14)
    load = gen.random_loads((2, 9, 9), seed=35, mean=6.0)
    _check(dyn, prof, sp, load, max_exempt=0.03)


def test_classes_with_and_without_load_thresholds_side_by_side(dyn):
    """A few table rows (classes 0, 4 and 8) cross the SLO twice: tiles of those classes take the general path, the
    other six classes keep the threshold path, in the same launch."""
    from parity import tables_with_few_rows_without_threshold
    prof, sp0, bad = tables_with_few_rows_without_threshold(29)
    assert {c for c, _, _ in bad} == {0, 4, 8}
    sp = gen.make_space(sp0.f_cand_mhz, 6, 60.0, slo_ttft=0.8, slo_tbt=0.1, gpu_budget=14)
    load = gen.random_loads((2, 11, 9), seed=36, mean=6.0)
    _check(dyn, prof, sp, load, max_exempt=0.03)


@pytest.mark.parametrize("tps,n_max,budget", [((1, 2, 4, 8), 3, 5), ((1, 2, 4, 8), 9, 9), ((1, 2, 4, 8), 16, 16),
                                              ((1, 2, 4, 8), 20, 21), ((2, 8), 12, 24), ((1, 4, 8), 24, 24),
                                              ((1, 2, 4, 8), 24, 26)])
def test_list_lengths_around_the_chunk_and_kernel_limits(dyn, tps, n_max, budget):
    """Short tuple lists are evaluated as (tuple, TP index) pairs in chunks of 64 that may run over from one TP index
    into the next; lists beyond 512 tuples take the kernel that holds tuples in lanes.  Lists of 14 to about 900 tuples,
    with two to four parallelisms, cover chunks that are padded out, chunks that run over, and both kernels."""
    wl = gen.workload("cfg2")
    prof = gen.make_profile(tps, wl.f_grid_mhz, wl.M, gen.class_coefficients(7))
    sp = gen.make_space(wl.f_cand_mhz, n_max, wl.window_s, gpu_budget=budget)
    load = gen.random_loads((2, 24, 9), seed=71, mean=2.0)
    _check(dyn, prof, sp, load)
