"""GPU parity of the token-weighted loads (exact 64-bit sums, fp32 tokens per second bit for bit) and of the
carbon totals (fp64, 1e-12: the kernel adds the windows in a different fixed order than the oracle)."""
import numpy as np
import pytest
import torch

import gen
import oracle
from parity import dev_u32

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dyn():
    import paper_2408_00741_b200 as d
    assert torch.cuda.is_available()
    return d


def _gpu_tokens(dyn, t, a, b, wm, W, ie, oe, tps=True):
    Cn = (len(ie) + 1) * (len(oe) + 1)
    ti = torch.full((W, Cn), -1, dtype=torch.int64, device="cuda")
    to = torch.full((W, Cn), -1, dtype=torch.int64, device="cuda")
    lt = torch.full((W, Cn), -1.0, dtype=torch.float32, device="cuda") if tps else None
    dyn.dyn_bin_tokens(wm, W, ie, oe, dev_u32(t), dev_u32(a), dev_u32(b), ti, to, lt)
    torch.cuda.synchronize()
    return ti.cpu().numpy().view(np.uint64), to.cpu().numpy().view(np.uint64), (lt.cpu().numpy() if tps else None)


@pytest.mark.parametrize("name,scale", [("cfg1", 1.0), ("cfg2", 0.25), ("cfg3", 0.02)])
def test_token_sums_on_the_benchmark_traces(dyn, name, scale):
    wl = gen.workload(name, scale=scale)
    t, a, b = gen.make_trace(wl.trace)
    W = wl.trace.n_windows
    ti, to, lt = _gpu_tokens(dyn, t, a, b, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    ri, ro = oracle.bin_tokens(t, a, b, wl.trace.window_ms, W, gen.IN_EDGES, gen.OUT_EDGES)
    assert np.array_equal(ti, ri) and np.array_equal(to, ro)
    assert np.array_equal(lt, oracle.load_tps(ri, ro, wl.window_s))


def test_unsorted_sparse_huge_tokens_and_dropped_requests(dyn):
    rng = np.random.default_rng(8)
    n = 70_001                                              # several slices and a ragged tail
    t = rng.integers(0, 5_000_000, n).astype(np.uint32)     # unsorted, wide: most requests leave the CTA's window range
    a = rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32)      # sums far beyond 32 bits
    b = rng.integers(0, 2 ** 32, n, dtype=np.uint64).astype(np.uint32)
    ie, oe = np.array([1 << 20, 1 << 30], np.uint32), np.array([1 << 16], np.uint32)
    ti, to, _ = _gpu_tokens(dyn, t, a, b, 1000, 4000, ie, oe, tps=False)    # windows past 4000 are dropped
    ri, ro = oracle.bin_tokens(t, a, b, 1000, 4000, ie, oe)
    assert np.array_equal(ti, ri) and np.array_equal(to, ro)
    assert int(ri.max()) > 2 ** 32


@pytest.mark.parametrize("offset", [0, 1], ids=["aligned", "4-byte-aligned"])
@pytest.mark.parametrize("grid", ["3x3", "5x2"])
def test_sorted_trace_with_token_counts_beyond_16_bits(dyn, offset, grid):
    """A time-sorted dense trace (the path without per-request range tests) whose token counts mix values below and
    above 65536; arrays that start 4 bytes off a 16-byte boundary take the scalar loads."""
    rng = np.random.default_rng(10 + offset)
    n = 150_003
    t = np.sort(rng.integers(0, 90_000, n)).astype(np.uint32)
    a = np.where(rng.random(n) < 0.1, rng.integers(0, 2 ** 32, n, dtype=np.uint64), rng.integers(1, 8193, n)).astype(np.uint32)
    b = np.where(rng.random(n) < 0.1, rng.integers(0, 2 ** 32, n, dtype=np.uint64), rng.integers(1, 2049, n)).astype(np.uint32)
    if grid == "3x3":
        ie, oe = gen.IN_EDGES, gen.OUT_EDGES
    else:
        ie, oe = np.array([64, 256, 1024, 1 << 20], np.uint32), np.array([300], np.uint32)
    Cn, W = (len(ie) + 1) * (len(oe) + 1), 80               # windows 80..89 are dropped
    dt, da, db = (dev_u32(np.concatenate([np.zeros(offset, np.uint32), x]))[offset:] for x in (t, a, b))
    ti = torch.full((W, Cn), -1, dtype=torch.int64, device="cuda")
    to = torch.full((W, Cn), -1, dtype=torch.int64, device="cuda")
    dyn.dyn_bin_tokens(1000, W, ie, oe, dt, da, db, ti, to, None)
    torch.cuda.synchronize()
    ri, ro = oracle.bin_tokens(t, a, b, 1000, W, ie, oe)
    assert np.array_equal(ti.cpu().numpy().view(np.uint64), ri) and np.array_equal(to.cpu().numpy().view(np.uint64), ro)
    assert int(ri.max()) > 2 ** 32


def test_empty_trace_and_errors(dyn):
    z = torch.zeros(0, dtype=torch.int32, device="cuda")
    ti = torch.full((3, 9), 5, dtype=torch.int64, device="cuda")
    to = torch.full((3, 9), 5, dtype=torch.int64, device="cuda")
    dyn.dyn_bin_tokens(1000, 3, gen.IN_EDGES, gen.OUT_EDGES, z, z, z, ti, to, None)
    torch.cuda.synchronize()
    assert int(ti.abs().sum()) == 0 and int(to.abs().sum()) == 0
    with pytest.raises(dyn.DynError) as e:
        dyn.dyn_bin_tokens(0, 3, gen.IN_EDGES, gen.OUT_EDGES, z, z, z, ti, to, None)
    assert e.value.status == dyn.DYN_EINVAL


def test_carbon_matches_the_oracle_and_repeats_bit_for_bit(dyn):
    rng = np.random.default_rng(9)
    S, W = 37, 1441
    ew = rng.uniform(0, 800, (S, W))
    it = (300 + 150 * np.sin(np.arange(W) * 2 * np.pi / 1440)).astype(np.float32)    # a daily intensity curve
    d_ew, d_it = torch.from_numpy(ew).cuda(), torch.from_numpy(it).cuda()
    out1 = torch.zeros(S, dtype=torch.float64, device="cuda")
    out2 = torch.zeros(S, dtype=torch.float64, device="cuda")
    dyn.dyn_carbon(d_ew, d_it, out1)
    dyn.dyn_carbon(d_ew, d_it, out2)
    torch.cuda.synchronize()
    np.testing.assert_allclose(out1.cpu().numpy(), oracle.carbon(ew, it), rtol=1e-12)
    assert torch.equal(out1, out2)
