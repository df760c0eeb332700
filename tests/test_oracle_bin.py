"""Pins for the oracle's stage (a): classify + window + count (thresholds table, Sec. 3.1)."""
import os

import numpy as np
import pytest
from scipy.stats import norm

import gen
import oracle


def _read_thresholds(golden_dir):
    rows = []
    for line in open(os.path.join(golden_dir, "thresholds.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append(tuple(int(x) for x in line.split(";")))
    return rows


def test_threshold_table_boundaries(golden_dir):
    """Each printed threshold lands in the class the table's < / >= signs give it."""
    rows = _read_thresholds(golden_dir)
    tin = np.array([r[0] for r in rows], dtype=np.uint32)
    tout = np.array([r[1] for r in rows], dtype=np.uint32)
    t = np.arange(len(rows), dtype=np.uint32) * 1000           # one request per window
    counts, dropped = oracle.bin_trace(t, tin, tout, 1000, len(rows), gen.IN_EDGES, gen.OUT_EDGES)
    assert dropped == 0
    for w, r in enumerate(rows):
        expect = np.zeros(9, dtype=np.uint32)
        expect[r[2]] = 1
        assert (counts[w] == expect).all(), (r, counts[w])


def test_window_boundaries_and_dropped():
    wm, W = 5000, 4
    t = np.array([0, 4999, 5000, 9999, 10000, 19999, 20000, 4_000_000_000], dtype=np.uint32)
    one = np.ones_like(t)
    counts, dropped = oracle.bin_trace(t, one, one, wm, W, gen.IN_EDGES, gen.OUT_EDGES)
    assert counts[:, 0].tolist() == [2, 2, 1, 1]
    assert counts[:, 1:].sum() == 0
    assert dropped == 2                                         # t = 20000 and the far outlier


def test_counts_sum_and_permutation_invariance():
    wl = gen.workload("cfg1")
    t, i, o = gen.make_trace(wl.trace)
    counts, dropped = oracle.bin_trace(t, i, o, wl.trace.window_ms, wl.trace.n_windows, gen.IN_EDGES, gen.OUT_EDGES)
    assert int(counts.sum()) + dropped == len(t)
    perm = np.random.default_rng(3).permutation(len(t))
    c2, d2 = oracle.bin_trace(t[perm], i[perm], o[perm], wl.trace.window_ms, wl.trace.n_windows,
                              gen.IN_EDGES, gen.OUT_EDGES)
    assert d2 == dropped and (c2 == counts).all()
    # fewer windows than the trace covers: the tail is dropped, the head is unchanged
    c3, d3 = oracle.bin_trace(t, i, o, wl.trace.window_ms, 10, gen.IN_EDGES, gen.OUT_EDGES)
    assert (c3 == counts[:10]).all() and d3 == len(t) - int(counts[:10].sum())


@pytest.mark.parametrize("edges", [([256, 1024], [100, 350]), ([512], [200]), ([64, 256, 1024], [50, 100, 350, 700]),
                                   ([], [100])])
def test_against_library_histogram(edges):
    """Same counts from numpy's searchsorted + bincount (a library route that shares nothing)."""
    ie, oe = (np.array(e, dtype=np.uint32) for e in edges)
    rng = np.random.default_rng(11)
    n, wm, W = 5000, 700, 9
    t = np.sort(rng.integers(0, wm * W + 900, n)).astype(np.uint32)
    i = rng.integers(1, 3000, n).astype(np.uint32)
    o = rng.integers(1, 1200, n).astype(np.uint32)
    counts, dropped = oracle.bin_trace(t, i, o, wm, W, ie, oe)
    KO = len(oe) + 1
    Cn = (len(ie) + 1) * KO
    w = t // wm
    keep = w < W
    cls = np.searchsorted(ie, i, side="right") * KO + np.searchsorted(oe, o, side="right")
    ref = np.bincount((w[keep] * Cn + cls[keep]).astype(np.int64), minlength=W * Cn).reshape(W, Cn)
    assert (counts == ref).all()
    assert dropped == int((~keep).sum())


@pytest.mark.parametrize("name,fin,fout", [
    ("cfg1", (600.0, 1.0), (200.0, 0.8)),
    ("cfg3", (1000.0, 1.0), (250.0, 0.8)),
    ("cfg3code", (2000.0, 1.0), (30.0, 0.8)),
])
def test_class_fractions_match_lognormal_closed_form(name, fin, fout):
    """Generator + binning against the normal CDF: P(class) of a rounded lognormal, within 4.5 sigma."""
    wl = gen.workload(name)
    wl.trace.n_req = min(wl.trace.n_req, 400_000)
    t, i, o = gen.make_trace(wl.trace)
    counts, dropped = oracle.bin_trace(t, i, o, wl.trace.window_ms, wl.trace.n_windows, gen.IN_EDGES, gen.OUT_EDGES)
    n = len(t)
    assert dropped == 0

    def bucket_probs(median, sigma, edges):
        # rint(X) < e  <=>  X < e - 0.5
        cdf = [norm.cdf((np.log(e - 0.5) - np.log(median)) / sigma) for e in edges]
        return np.diff([0.0] + cdf + [1.0])

    p = np.outer(bucket_probs(*fin, gen.IN_EDGES.tolist()), bucket_probs(*fout, gen.OUT_EDGES.tolist())).ravel()
    got = counts.sum(axis=0) / n
    sig = np.sqrt(p * (1 - p) / n)
    assert (np.abs(got - p) <= 4.5 * sig + 1e-9).all(), (got, p)
    # marginals of the 1-hour configuration, from the normal CDF by hand
    if name == "cfg1":
        pin = bucket_probs(*fin, gen.IN_EDGES.tolist())
        assert np.allclose(pin, [0.1972, 0.5063, 0.2965], atol=2e-3)


def test_load_is_count_over_window_in_fp32():
    counts = np.array([[0, 1, 59, 60, 61, 1389, 4_000_000]], dtype=np.uint32)
    ld = oracle.load_from_counts(counts, 60.0)
    assert ld.dtype == np.float32
    assert ld[0, 0] == 0.0 and ld[0, 3] == 1.0
    assert (ld == (counts.astype(np.float32) / np.float32(60.0))).all()
    ld5 = oracle.load_from_counts(counts, 5.0)
    assert ld5[0, 1] == np.float32(0.2)
