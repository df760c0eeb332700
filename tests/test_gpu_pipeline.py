"""GPU parity of the host-buffer entry point (copy in, bin, evaluate+select, totals, copy out)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import REL_TOL, check_selection

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


@pytest.mark.parametrize("name,S,pinned", [("cfg1", 1, False), ("cfg1", 3, True), ("cfg2", 2, True)])
def test_pipeline_host_matches_oracle(dyn, name, S, pinned):
    wl = gen.workload(name)
    t, i, o = gen.make_trace(wl.trace)
    prof, sp = wl.profile(), wl.space()
    W, Cn, J = wl.trace.n_windows, 9, wl.J
    ref_c, ref_d = oracle.bin_trace(t, i, o, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    extra = None
    if S > 1:
        cs = gen.resample_counts(ref_c, S - 1, seed=4, s_begin=1)
        extra = oracle.load_from_counts(cs, wl.window_s)
    SP = dyn.Space(sp.f_cand_mhz, sp.n_max, sp.slo_ttft_s, sp.slo_tbt_s, sp.window_s, sp.gpu_budget)
    hp = dyn.HostPipeline(wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES, prof.tp, prof.f_grid_mhz, prof.ttft,
                          prof.cap, prof.tbt, prof.pow, SP)
    mk = (lambda *shape, dtype: torch.empty(shape, dtype=dtype).pin_memory()) if pinned else \
         (lambda *shape, dtype: torch.empty(shape, dtype=dtype))
    out = {"counts": mk(W, Cn, dtype=torch.int32), "dropped": mk(1, dtype=torch.int64),
           "best_idx": mk(S, W, Cn, dtype=torch.int32), "best_E": mk(S, W, Cn, dtype=torch.float32),
           "E_total": mk(S, dtype=torch.float64), "n_infeasible": mk(S, dtype=torch.int32),
           "E_window": mk(S, W, dtype=torch.float64), "hist": mk(S, J, dtype=torch.int32),
           "gpus": mk(S, W, dtype=torch.int32)}
    nb = hp.arena_bytes(len(t), S)
    assert nb > 0 and nb % 256 == 0
    arena = torch.empty(nb, dtype=torch.uint8, device="cuda")
    for _ in range(2):                                      # the arena is reusable as is
        hp.run(t.view(np.int32), i.view(np.int32), o.view(np.int32), extra, out, arena)
        torch.cuda.synchronize()
    assert np.array_equal(out["counts"].numpy().view(np.uint32), ref_c)
    assert int(out["dropped"].item()) == ref_d
    load0 = oracle.load_from_counts(ref_c, wl.window_s)[None]
    load = load0 if extra is None else np.concatenate([load0, extra])
    ref = oracle.eval_select(prof, sp, load)
    fixed, _ = check_selection(prof, sp, load, out["best_idx"].numpy(), out["best_E"].numpy(), ref)
    nj, tj = oracle.config_tables(sp.n_max, prof.tp, sp.F)
    tot = oracle.totals(ref["best_idx"], ref["best_E"], J, nj, tj)
    assert np.allclose(out["E_total"].numpy(), tot["E_total"], rtol=REL_TOL)
    assert np.allclose(out["E_window"].numpy(), tot["E_window"], rtol=REL_TOL, atol=1e-12)
    assert np.array_equal(out["n_infeasible"].numpy().astype(np.int64), tot["n_infeasible"].astype(np.int64))
    assert int(out["hist"].numpy().sum()) == load.size - int(tot["n_infeasible"].sum())
    # a short arena is refused before anything is enqueued
    with pytest.raises(dyn.DynError) as e:
        hp.run(t.view(np.int32), i.view(np.int32), o.view(np.int32), extra, out, arena[:nb - 256])
    assert e.value.status == dyn.DYN_EWORKSPACE


@pytest.mark.parametrize("S", [2, 12, 40])
def test_copy_stream_gives_the_same_results(dyn, S):
    """With a second stream the scenario loads arrive in pieces (here fewer and more scenarios than pieces), every
    piece is evaluated on its own and its results are copied back on the second stream: all outputs equal those of
    the single-stream call bit for bit, and waiting for the caller's stream alone is enough to read them."""
    wl = gen.workload("cfg1")
    t, i, o = gen.make_trace(wl.trace)
    prof, sp = wl.profile(), wl.space()
    W, Cn, J = wl.trace.n_windows, 9, wl.J
    ref_c, _ = oracle.bin_trace(t, i, o, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    extra = torch.from_numpy(oracle.load_from_counts(gen.resample_counts(ref_c, S - 1, seed=4, s_begin=1),
                                                     wl.window_s)).pin_memory()
    SP = dyn.Space(sp.f_cand_mhz, sp.n_max, sp.slo_ttft_s, sp.slo_tbt_s, sp.window_s, sp.gpu_budget)
    hp = dyn.HostPipeline(wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES, prof.tp, prof.f_grid_mhz, prof.ttft,
                          prof.cap, prof.tbt, prof.pow, SP)

    def buffers():
        mk = lambda *shape, dtype: torch.zeros(shape, dtype=dtype).pin_memory()
        return {"counts": mk(W, Cn, dtype=torch.int32), "best_idx": mk(S, W, Cn, dtype=torch.int32),
                "best_E": mk(S, W, Cn, dtype=torch.float32), "E_total": mk(S, dtype=torch.float64),
                "n_infeasible": mk(S, dtype=torch.int32), "E_window": mk(S, W, dtype=torch.float64),
                "hist": mk(S, J, dtype=torch.int32), "gpus": mk(S, W, dtype=torch.int32)}

    arena = torch.empty(hp.arena_bytes(len(t), S), dtype=torch.uint8, device="cuda")
    one, two = buffers(), buffers()
    hp.run(t.view(np.int32), i.view(np.int32), o.view(np.int32), extra, one, arena)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    for _ in range(2):                                      # back to back: the second call waits for the first one's use of the arena
        hp.run(t.view(np.int32), i.view(np.int32), o.view(np.int32), extra, two, arena, copy_stream=side)
    torch.cuda.current_stream().synchronize()               # not the copy stream: the call orders it before this one
    for k in one:
        assert torch.equal(one[k], two[k]), k
