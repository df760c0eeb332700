"""Whole path on tiny grids against an independent restatement built on numpy.interp and Python
dicts: trace -> counts -> loads -> every candidate -> choice -> totals."""
import numpy as np
import pytest

import gen
import oracle


def _brute(t_ms, tin, tout, wm, W, ie, oe, prof, sp):
    KO = len(oe) + 1
    Cn = (len(ie) + 1) * KO
    counts = {}
    for t, a, b in zip(t_ms.tolist(), tin.tolist(), tout.tolist()):
        w = t // wm
        if w >= W:
            continue
        c = sum(1 for e in ie.tolist() if e <= a) * KO + sum(1 for e in oe.tolist() if e <= b)
        counts[(w, c)] = counts.get((w, c), 0) + 1
    fg = prof.f_grid_mhz.astype(np.float64)
    M = prof.M
    uk = np.arange(M) / (M - 1)
    out = {}
    for w in range(W):
        for c in range(Cn):
            L = float(np.float32(counts.get((w, c), 0)) / np.float32(sp.window_s))
            best, bj = np.inf, -1
            j = 0
            for n in range(1, sp.n_max + 1):
                for t in range(prof.T):
                    for q in range(sp.F):
                        f = float(sp.f_cand_mhz[q])
                        ttft = np.interp(f, fg, prof.ttft[c, t].astype(np.float64))
                        cap = np.interp(f, fg, prof.cap[c, t].astype(np.float64))
                        u = L / n / cap
                        uc = min(u, 1.0)
                        tb_rows = [np.interp(uc, uk, prof.tbt[c, t, r].astype(np.float64)) for r in range(prof.R)]
                        pw_rows = [np.interp(uc, uk, prof.pow[c, t, r].astype(np.float64)) for r in range(prof.R)]
                        tbt = np.interp(f, fg, tb_rows)
                        pw = np.interp(f, fg, pw_rows)
                        ok = ttft <= sp.slo_ttft_s[c] and tbt <= sp.slo_tbt_s[c] and u <= 1.0
                        if sp.gpu_budget > 0 and n * int(prof.tp[t]) > sp.gpu_budget:
                            ok = False
                        E = n * pw * sp.window_s / 3600.0 if ok else np.inf
                        if E < best:
                            best, bj = E, j
                        j += 1
            out[(w, c)] = (bj, best)
    return counts, out


@pytest.mark.parametrize("budget", [0, 6])
def test_tiny_grid_brute_force(budget):
    rng = np.random.default_rng(21)
    ie, oe = np.array([300], np.uint32), np.array([120], np.uint32)        # C = 4
    wm, W, n = 2000, 2, 60
    t_ms = np.sort(rng.integers(0, wm * W + 500, n)).astype(np.uint32)
    tin = rng.integers(1, 900, n).astype(np.uint32)
    tout = rng.integers(1, 400, n).astype(np.uint32)
    Cn, T, R, M, F, N = 4, 2, 4, 3, 3, 3
    tp = np.array([2, 4], np.int32)
    fg = np.array([800, 1100, 1500, 1980], np.float32)
    ttft = (0.2 + rng.random((Cn, T, R))).astype(np.float32)
    cap = (4.0 + 6.0 * rng.random((Cn, T, R))).astype(np.float32)
    tbt = np.sort(0.02 + 0.12 * rng.random((Cn, T, R, M)), axis=-1).astype(np.float32)
    pw = (200 + 500 * rng.random((Cn, T, R, M))).astype(np.float32)         # deliberately not monotone
    prof = gen.Profile(tp, fg, ttft, cap, tbt, pw)
    sp = gen.make_space(np.array([800, 1300, 1980], np.float32), N, wm / 1000.0, C=Cn,
                        slo_ttft=1.0, slo_tbt=0.1, gpu_budget=budget)

    counts, dropped = oracle.bin_trace(t_ms, tin, tout, wm, W, ie, oe)
    ref_counts, ref = _brute(t_ms, tin, tout, wm, W, ie, oe, prof, sp)
    for w in range(W):
        for c in range(Cn):
            assert counts[w, c] == ref_counts.get((w, c), 0)
    assert dropped == n - sum(ref_counts.values())
    load = oracle.load_from_counts(counts, sp.window_s)
    r = oracle.eval_select(prof, sp, load[None])
    n_feasible = 0
    for w in range(W):
        for c in range(Cn):
            bj, be = ref[(w, c)]
            assert r["best_idx"][0, w, c] == bj
            if bj >= 0:
                n_feasible += 1
                assert r["best_E"][0, w, c] == pytest.approx(be, rel=1e-12)
    assert n_feasible >= 4
    tot = oracle.totals(r["best_idx"], r["best_E"], N * T * F)
    assert tot["E_total"][0] == pytest.approx(sum(e for j, e in ref.values() if j >= 0), rel=1e-12)
