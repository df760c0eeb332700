"""GPU parity of the hierarchical selection (Sec. 4.2) against the oracle: nodes, sharding and the
per-window choice identical except where a deciding quantity or an energy gap is within 1e-5."""
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


def _run(dyn, prof, sp, e1, e2, load):
    S, W, Cn = load.shape
    J = sp.n_max * prof.T * sp.F
    K1, K2 = -(-W // e1), -(-W // e2)
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load).cuda()
    nodes = torch.full((S, K1, Cn), -7, dtype=torch.int32, device="cuda")
    shard = torch.full((S, K2, Cn), -7, dtype=torch.int32, device="cuda")
    out = dyn.SelectOut(S, W, Cn, J)
    ws = torch.empty(dyn.dyn_hier_workspace_bytes(p, s, S, W), dtype=torch.uint8, device="cuda")
    dyn.dyn_hier_select(p, s, e1, e2, d_load, nodes, shard, out, ws)
    torch.cuda.synchronize()
    return nodes.cpu().numpy(), shard.cpu().numpy(), out


def _check(dyn, prof, sp, e1, e2, load, max_exempt=0.01):
    S, W, Cn = load.shape
    ref = oracle.hier_select(prof, sp, e1, e2, load)
    nodes, shard, out = _run(dyn, prof, sp, e1, e2, load)
    idx, E = out.best_idx.cpu().numpy(), out.best_E.cpu().numpy()
    # nodes: exact unless PL/ML sits on an integer
    frac = ref["nodes_frac"]
    with np.errstate(invalid="ignore"):                     # inf - inf where a class has no feasible load at all
        n_ex = np.abs(frac - np.rint(frac)) < REL_TOL
    assert ((nodes == ref["nodes"]) | n_ex).all()
    # sharding: exact unless its own decision is near a bound / a tie, or its nodes were exempt
    up1 = np.repeat(n_ex, e1 // e2, axis=1)[:, :shard.shape[1]]
    s_ex = up1 | (ref["shard_margin"] < REL_TOL) | (ref["shard_gap"] < REL_TOL)
    assert ((shard == ref["shard"]) | s_ex).all()
    # windows
    up2 = np.repeat(s_ex, e2, axis=1)[:, :W]
    t_ex = up2 | (ref["freq_margin"] < REL_TOL) | (ref["freq_gap"] < REL_TOL)
    same = idx == ref["best_idx"]
    assert (same | t_ex).all()
    assert (~same).sum() <= max(3, max_exempt * same.size)   # exempted tiles may differ, but few do
    ok = same & (ref["best_idx"] >= 0)
    rel = np.abs(E[ok].astype(np.float64) - ref["best_E"][ok]) / ref["best_E"][ok]
    assert rel.max() <= REL_TOL
    assert np.isinf(E[same & (ref["best_idx"] < 0)]).all()
    # totals of the GPU's own choice
    fin = np.where(idx >= 0, E.astype(np.float64), 0.0).sum(axis=(1, 2))
    assert np.allclose(out.E_total.cpu().numpy(), fin, rtol=1e-9)
    assert np.array_equal(out.n_infeasible.cpu().numpy(), (idx < 0).sum(axis=(1, 2)))
    return ref, idx, E


@pytest.mark.parametrize("name,W,e1,e2,mean", [("cfg1", 60, 30, 5, 3.0), ("cfg2", 97, 12, 4, 6.0), ("cfg2", 40, 1, 1, 2.5),
                                               ("cfg3", 64, 64, 64, 2.0), ("cfg5", 6, 6, 2, 2.0)])
def test_hier_select_matches_oracle(dyn, name, W, e1, e2, mean):
    wl = gen.workload(name)
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((2, W, 9), seed=21, mean=mean)
    load[0, 0] = 0.0
    ref, idx, E = _check(dyn, prof, sp, e1, e2, load)
    assert (ref["best_idx"] >= 0).mean() > 0.5


def test_hier_with_gpu_budget_and_infeasible_pools(dyn):
    wl = gen.workload("cfg2")
    prof = wl.profile()
    sp = gen.make_space(wl.f_cand_mhz, wl.n_max, wl.window_s, gpu_budget=16)
    load = gen.random_loads((1, 36, 9), seed=5, mean=8.0)
    load[0, 12:24, 3] = 500.0                               # more than 16 GPUs can serve
    ref, idx, E = _check(dyn, prof, sp, 12, 6, load)
    assert (idx[0, 12:24, 3] == -1).all()


def test_hier_energy_is_never_below_the_joint_optimum(dyn):
    wl = gen.workload("cfg2")
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((2, 60, 9), seed=8, mean=3.0)
    nodes, shard, out = _run(dyn, prof, sp, 30, 5, load)
    from parity import gpu_eval_select
    joint = gpu_eval_select(dyn, prof, sp, load)
    Eh, Ej = out.best_E.cpu().numpy().astype(np.float64), joint.best_E.cpu().numpy().astype(np.float64)
    both = np.isfinite(Eh) & np.isfinite(Ej)
    assert (Eh[both] >= Ej[both] * (1 - 1e-6)).all()
    assert float(out.E_total.sum()) > float(joint.E_total.sum())


def test_hier_argument_errors(dyn):
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((1, 8, 9), seed=1)
    with pytest.raises(dyn.DynError) as e:
        _run(dyn, prof, sp, 5, 2, load)
    assert e.value.status == dyn.DYN_EINVAL


@pytest.mark.parametrize("large", [False, True], ids=["tables-in-shared-memory", "tables-through-L1"])
@pytest.mark.parametrize("monotone", [False, True], ids=["tbt-rises-and-falls", "tbt-never-decreases"])
def test_hier_free_form_tables(dyn, monotone, large):
    """Both variants of the sharding and frequency kernels: the threshold variants need every TBT row monotone and
    tables that fit in shared memory; otherwise the plain variants evaluate from the general-path tables."""
    from parity import random_tables
    prof, sp = random_tables(29, monotone, large)
    load = gen.random_loads((2, 24, 9), seed=36, mean=5.0)
    _check(dyn, prof, sp, 12, 4, load, max_exempt=0.03)


def test_hier_classes_with_and_without_load_thresholds(dyn):
    """A few table rows (classes 0, 4 and 8) cross the SLO twice: the warps of those classes evaluate from the
    general-path tables, the other six classes keep the threshold path, in the same launches."""
    from parity import tables_with_few_rows_without_threshold
    prof, sp, bad = tables_with_few_rows_without_threshold(31)
    assert {c for c, _, _ in bad} == {0, 4, 8}
    load = gen.random_loads((2, 24, 9), seed=37, mean=5.0)
    _check(dyn, prof, sp, 12, 4, load, max_exempt=0.03)


@pytest.mark.parametrize("shape", ["convex", "concave", "falling"])
def test_hier_energy_rows_that_are_not_lines(dyn, shape):
    """The sharding level stops its walk over the counts on a line under the degree's energy row.  Rows that bend
    upwards (the line's intercept is negative: no early stop at that degree), bend downwards, or fall with the load
    must give the choices of the full walk, which the oracle does."""
    import dataclasses
    wl = gen.workload("cfg2")
    prof, sp = wl.profile(), wl.space()
    u = np.linspace(0.0, 1.0, prof.M, dtype=np.float64)
    tp = prof.tp.astype(np.float64)[None, :, None, None]
    s3 = (prof.f_grid_mhz.astype(np.float64) / 1980.0)[None, None, :, None] ** 3
    if shape == "convex":
        pw = 5.0 * tp + 900.0 * tp * s3 * u ** 3
    elif shape == "concave":
        pw = 120.0 * tp + 500.0 * tp * s3 * np.sqrt(u)
    else:
        pw = 700.0 * tp - 450.0 * tp * s3 * u
    pw = np.broadcast_to(pw, prof.pow.shape).astype(np.float32).copy()
    prof = dataclasses.replace(prof, pow=pw)
    load = gen.random_loads((2, 48, 9), seed=41, mean=4.0)
    load[1, :, 2] *= 6.0                                     # a class that needs many instances
    _check(dyn, prof, sp, 12, 4, load, max_exempt=0.03)
