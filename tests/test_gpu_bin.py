"""GPU parity, stage (a): counts bit-exact against the oracle, loads bit-exact (one fp32 divide)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import dev_u32, gpu_bin_trace

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _check(dyn, t, i, o, wm, W, ie=gen.IN_EDGES, oe=gen.OUT_EDGES, **kw):
    ref_c, ref_d = oracle.bin_trace(t, i, o, wm, W, ie, oe)
    got_c, got_l, got_d = gpu_bin_trace(dyn, t, i, o, wm, W, ie, oe, **kw)
    assert got_d == ref_d
    assert np.array_equal(got_c, ref_c)
    assert int(got_c.sum()) + got_d == len(t)
    if got_l is not None:
        assert np.array_equal(got_l, oracle.load_from_counts(ref_c, np.float32(wm) / np.float32(1000.0)))
    return ref_c


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg3code"])
def test_benchmark_traces_full_size(dyn, name):
    wl = gen.workload(name)
    t, i, o = gen.make_trace(wl.trace)
    _check(dyn, t, i, o, wl.trace.window_ms, wl.trace.n_windows)


@pytest.mark.parametrize("n", [0, 1, 31, 127, 128, 129, 1000, 4097, 100_003])
def test_ragged_sizes(dyn, n):
    rng = np.random.default_rng(n)
    wm, W = 250, 37
    t = np.sort(rng.integers(0, wm * W + 300, n)).astype(np.uint32)
    i = rng.integers(1, 3000, n).astype(np.uint32)
    o = rng.integers(1, 1200, n).astype(np.uint32)
    _check(dyn, t, i, o, wm, W)


def test_unsorted_trace_and_few_windows(dyn):
    wl = gen.workload("cfg2", scale=0.05)
    t, i, o = gen.make_trace(wl.trace)
    perm = np.random.default_rng(1).permutation(len(t))
    _check(dyn, t[perm], i[perm], o[perm], wl.trace.window_ms, wl.trace.n_windows)
    _check(dyn, t[perm], i[perm], o[perm], wl.trace.window_ms, 5)           # most requests dropped
    _check(dyn, t, i, o, 86_400_000, 1)                                     # one window


@pytest.mark.parametrize("n,per_window", [(3_000_000, 0.7), (20_000_000, 12.0), (45_000_000, 40.0)])
def test_long_sparse_trace(dyn, n, per_window):
    """Many windows per request slice: a CTA's slice no longer fits its shared-memory bins and is taken in
    pieces (long slices, 12 requests per window) or spills to global atomics (fewer than one per window); with
    45 M requests the grid grows so that a slice stays at about 24 K requests."""
    rng = np.random.default_rng(7)
    W = int(n / per_window)
    wm = 3
    t = np.sort(rng.integers(0, W * wm, n)).astype(np.uint32)
    i = rng.integers(1, 3000, n).astype(np.uint32)
    o = rng.integers(1, 1200, n).astype(np.uint32)
    _check(dyn, t, i, o, wm, W)


def test_window_edges_and_large_timestamps(dyn):
    for wm in (1, 7, 1000, 5000, 60_000, 65_536, 86_400_000, 4_294_967_295):
        ks = np.arange(0, 40, dtype=np.uint64)
        t = np.concatenate([ks * wm, ks * wm + (wm - 1), [4_294_967_295, 4_294_967_294, 2_147_483_648]])
        t = np.sort(t[t < 2 ** 32]).astype(np.uint32)
        one = np.full(len(t), 300, dtype=np.uint32)
        _check(dyn, t, one, one, wm, 40)
        _check(dyn, t, one, one, wm, 65_000 if wm > 60_000 else 40)


def test_threshold_values(dyn):
    tin = np.array([255, 256, 1023, 1024, 8192, 1, 0, 4_000_000_000], dtype=np.uint32)
    tout = np.array([99, 100, 349, 350, 8192, 1, 0, 4_000_000_000], dtype=np.uint32)
    ii, oo = np.meshgrid(tin, tout, indexing="ij")
    n = ii.size
    t = (np.arange(n) * 10).astype(np.uint32)
    _check(dyn, t, ii.ravel(), oo.ravel(), 100, 7)


@pytest.mark.parametrize("edges", [([512], [200]), ([], []), ([64, 256, 1024], [50, 100, 350]),
                                   ([64, 256, 1024], [50, 100, 350, 700]),
                                   (list(range(100, 1600, 100)), list(range(50, 800, 50)))])
def test_other_class_grids(dyn, edges):
    """2, 1, 16, 20 and 256 classes: packed-counter path up to 16 classes, leader-election path above."""
    ie, oe = (np.array(e, dtype=np.uint32) for e in edges)
    wl = gen.workload("cfg2", scale=0.02)
    t, i, o = gen.make_trace(wl.trace)
    _check(dyn, t, i, o, wl.trace.window_ms, wl.trace.n_windows, ie, oe)
    perm = np.random.default_rng(2).permutation(len(t))
    _check(dyn, t[perm], i[perm], o[perm], wl.trace.window_ms, wl.trace.n_windows, ie, oe)


def test_unaligned_device_arrays_and_no_load_output(dyn):
    wl = gen.workload("cfg1")
    t, i, o = gen.make_trace(wl.trace)
    pad = lambda x: dev_u32(np.concatenate([[0], x]))[1:]                   # 4-byte aligned only
    _check(dyn, t, i, o, wl.trace.window_ms, wl.trace.n_windows, device_arrays=(pad(t), pad(i), pad(o)),
           want_load=False)


def test_argument_errors(dyn):
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    cnt = torch.zeros((2, 9), dtype=torch.int32, device="cuda")
    dr = torch.zeros(1, dtype=torch.int64, device="cuda")
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_bin_trace(0, 2, gen.IN_EDGES, gen.OUT_EDGES, z, z, z, cnt, None, dr)
    assert e.value.status == dyn.DYN_EINVAL
    with pytest.raises(dyn.DynError):
        dyn.dyn_bin_trace(10, 2, [1024, 256], gen.OUT_EDGES, z, z, z, cnt, None, dr)      # edges not ascending
    with pytest.raises(dyn.DynError):
        dyn.dyn_bin_trace(10, 2, list(range(1, 18)), gen.OUT_EDGES, z, z, z, cnt, None, dr)  # too many edges
    with pytest.raises(dyn.DynError):
        dyn.dyn_bin_trace(10, 0, gen.IN_EDGES, gen.OUT_EDGES, z, z, z, cnt, None, dr)
