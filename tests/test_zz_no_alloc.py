"""dyn_eval_select_static: the entry point for callers that cannot allocate device memory (a guest
controller inside a serving process that owns the whole GPU, a plug-in barred from the CUDA allocator).
It must give what dyn_eval_select gives with a caller workspace, call after call, although all calls
share one fixed scratch array that still holds the previous call's tables."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import check_selection, gpu_profile_space

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _both(dyn, wl, S, W, seed):
    prof, sp = wl.profile(), wl.space()
    load = gen.random_loads((S, W, 9), seed=seed, mean=2.5)
    load[0, 0, :] = 0.0
    load[0, 1, :] = 1e4                                    # no feasible candidate
    p, s = gpu_profile_space(dyn, prof, sp)
    d_load = torch.from_numpy(load).cuda()
    ref = dyn.SelectOut(S, W, 9, wl.J)
    ws = torch.empty(dyn.dyn_workspace_bytes(p, s, S, W), dtype=torch.uint8, device="cuda")
    dyn.dyn_eval_select(p, s, d_load, ref, ws)             # existing entry point, caller workspace
    got = dyn.SelectOut(S, W, 9, wl.J)
    for t in (got.best_idx, got.n_infeasible, got.hist, got.gpus):
        t.fill_(-12345)
    dyn.dyn_eval_select_static(p, s, d_load, got)          # new entry point, no workspace
    torch.cuda.synchronize()
    # and against the CPU oracle directly, under the rule of the other parity tests
    o = oracle.eval_select(prof, sp, load)
    check_selection(prof, sp, load, got.best_idx.cpu().numpy(), got.best_E.cpu().numpy(), o)
    return ref, got


def _same(ref, got):
    assert torch.equal(ref.best_idx, got.best_idx)
    e_ref, e_got = ref.best_E.cpu().numpy().astype(np.float64), got.best_E.cpu().numpy().astype(np.float64)
    fin = np.isfinite(e_ref)
    assert np.array_equal(fin, np.isfinite(e_got))
    assert np.allclose(e_got[fin], e_ref[fin], rtol=1e-5, atol=0)
    assert np.allclose(got.E_total.cpu().numpy(), ref.E_total.cpu().numpy(), rtol=1e-5)
    assert np.allclose(got.E_window.cpu().numpy(), ref.E_window.cpu().numpy(), rtol=1e-5, atol=1e-12)
    assert torch.equal(ref.n_infeasible, got.n_infeasible)
    assert torch.equal(ref.hist, got.hist) and torch.equal(ref.gpus, got.gpus)
    assert int((got.best_idx >= 0).sum()) > 0 and int((got.best_idx < 0).sum()) >= 9


def test_static_scratch_matches_workspace_variant_twice_in_a_row(dyn):
    # two different problems back to back: the second call finds the first one's tables in the scratch
    ref, got = _both(dyn, gen.workload("cfg1"), S=2, W=50, seed=21)
    _same(ref, got)
    ref, got = _both(dyn, gen.workload("cfg2"), S=3, W=40, seed=22)
    _same(ref, got)
    # and the first problem again, after the larger one
    ref, got = _both(dyn, gen.workload("cfg1"), S=1, W=17, seed=23)
    _same(ref, got)


def test_problem_larger_than_the_static_scratch_is_refused(dyn):
    wl = gen.workload("cfg5")
    prof = gen.make_profile(wl.tp, np.array([800.0, 1980.0], np.float32), 160, gen.class_coefficients(5))
    sp = wl.space()
    p, s = gpu_profile_space(dyn, prof, sp)
    assert dyn.dyn_workspace_bytes(p, s, 1, 2) > dyn.DYN_STATIC_WS_BYTES
    out = dyn.SelectOut(1, 2, 9, wl.J)
    out.best_idx.fill_(7)
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select_static(p, s, torch.zeros((1, 2, 9), dtype=torch.float32, device="cuda"), out)
    assert e.value.status == dyn.DYN_EUNSUPPORTED
    torch.cuda.synchronize()
    assert int((out.best_idx == 7).sum()) == 18            # nothing was enqueued
    # the same problem is served by the workspace variant
    ws = torch.empty(dyn.dyn_workspace_bytes(p, s, 1, 2), dtype=torch.uint8, device="cuda")
    dyn.dyn_eval_select(p, s, torch.zeros((1, 2, 9), dtype=torch.float32, device="cuda"), out, ws)
    torch.cuda.synchronize()
    assert int((out.best_idx == 7).sum()) < 18


def test_largest_problem_that_fits_and_no_allocation(dyn):
    """A problem whose scratch need is within 256 bytes of the static array is served, the next larger one is
    refused; and a call changes nothing in the device's free memory (it allocates nothing)."""
    wl = gen.workload("cfg1")
    prof, sp = wl.profile(), wl.space()
    p, s = gpu_profile_space(dyn, prof, sp)
    W = 1
    lo, hi = 1, 1 << 22
    while lo < hi:                                          # largest S whose workspace fits
        mid = (lo + hi + 1) // 2
        if dyn.dyn_workspace_bytes(p, s, mid, W) <= dyn.DYN_STATIC_WS_BYTES:
            lo = mid
        else:
            hi = mid - 1
    S = lo
    need = dyn.dyn_workspace_bytes(p, s, S, W)
    assert dyn.DYN_STATIC_WS_BYTES - 256 <= need <= dyn.DYN_STATIC_WS_BYTES
    load = gen.random_loads((S, W, 9), seed=31, mean=2.5)
    d_load = torch.from_numpy(load).cuda()
    got = dyn.SelectOut(S, W, 9, wl.J, windows=False, hist=False, gpus=False)
    ref = dyn.SelectOut(S, W, 9, wl.J, windows=False, hist=False, gpus=False)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    dyn.dyn_eval_select_static(p, s, d_load, got)           # (also the warm-up call of this device, if none came before)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    dyn.dyn_eval_select_static(p, s, d_load, got)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    dyn.dyn_eval_select(p, s, d_load, ref, ws)
    torch.cuda.synchronize()
    assert torch.equal(ref.best_idx, got.best_idx) and torch.equal(ref.n_infeasible, got.n_infeasible)
    assert np.allclose(got.E_total.cpu().numpy(), ref.E_total.cpu().numpy(), rtol=1e-5)
    # one scenario block more no longer fits
    S2 = S + 64
    assert dyn.dyn_workspace_bytes(p, s, S2, W) > dyn.DYN_STATIC_WS_BYTES
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_eval_select_static(p, s, torch.zeros((S2, W, 9), dtype=torch.float32, device="cuda"),
                                   dyn.SelectOut(S2, W, 9, wl.J, windows=False, hist=False, gpus=False))
    assert e.value.status == dyn.DYN_EUNSUPPORTED
