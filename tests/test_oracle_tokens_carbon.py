"""Pins of the oracle's token-weighted loads and carbon: numpy's weighted bincount, conservation of tokens,
agreement with the request counts on unit tokens, and numpy's dot product."""
import numpy as np

import gen
import oracle


def _trace(n=5000, seed=3):
    rng = np.random.default_rng(seed)
    t = np.sort(rng.integers(0, 70_000, n)).astype(np.uint32)          # some past the last window
    a = rng.integers(1, 9000, n).astype(np.uint32)
    b = rng.integers(1, 2000, n).astype(np.uint32)
    return t, a, b


def test_token_sums_against_weighted_bincount():
    t, a, b = _trace()
    wm, W = 1000, 60
    ti, to = oracle.bin_tokens(t, a, b, wm, W, gen.IN_EDGES, gen.OUT_EDGES)
    w = t // wm
    c = np.searchsorted(gen.IN_EDGES, a, side="right") * 3 + np.searchsorted(gen.OUT_EDGES, b, side="right")
    keep = w < W
    flat = (w[keep].astype(np.int64) * 9 + c[keep])
    for got, tok in ((ti, a), (to, b)):
        want = np.zeros(W * 9, np.uint64)
        np.add.at(want, flat, tok[keep].astype(np.uint64))
        assert np.array_equal(got.ravel(), want)
    assert int(ti.sum()) == int(a[keep].astype(np.uint64).sum()) and int(to.sum()) == int(b[keep].astype(np.uint64).sum())
    assert (~keep).any()


def test_unit_tokens_give_the_request_counts_and_large_tokens_do_not_wrap():
    t, a, b = _trace(seed=4)
    counts, _ = oracle.bin_trace(t, a, b, 1000, 60, gen.IN_EDGES, gen.OUT_EDGES)
    # classes depend on the token values, so count with the real tokens and weight with ones via a second call
    ones = np.ones_like(a)
    ti, _ = oracle.bin_tokens(t, ones, ones, 1000, 60, np.array([], np.uint32), np.array([], np.uint32))
    assert np.array_equal(ti[:, 0], counts.sum(axis=1).astype(np.uint64))
    big = np.full(8, 0xFFFFFFFF, np.uint32)
    ti, to = oracle.bin_tokens(np.zeros(8, np.uint32), big, big, 10, 1, gen.IN_EDGES, gen.OUT_EDGES)
    assert int(ti[0, 8]) == 8 * 0xFFFFFFFF and int(to[0, 8]) == 8 * 0xFFFFFFFF      # beyond 32 bits


def test_tokens_per_second_rounding():
    ti = np.array([[3, 1 << 40]], np.uint64)
    to = np.array([[4, 5]], np.uint64)
    tps = oracle.load_tps(ti, to, 60.0)
    assert tps.dtype == np.float32
    assert tps[0, 0] == np.float32(7) / np.float32(60) and tps[0, 1] == np.float32((1 << 40) + 5) / np.float32(60)


def test_carbon_is_the_dot_product():
    rng = np.random.default_rng(5)
    ew = rng.uniform(0, 500, (4, 288))
    it = rng.uniform(100, 500, 288).astype(np.float32)
    got = oracle.carbon(ew, it)
    np.testing.assert_allclose(got, ew @ it.astype(np.float64) / 1000.0, rtol=1e-13)
    assert oracle.carbon(np.ones((1, 3)), np.array([1000, 0, 500], np.float32))[0] == 1.5
