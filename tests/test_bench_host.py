"""Host-side logic of the benchmark: the max-over-ranks reduction (2 gloo ranks on CPU), the oracle
step used by the CPU-baseline and reference arms, and the clock-sample parser."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    got = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    q.put((rank, got))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    ps = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in ps:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in ps:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, 15.0), (1, 15.0)]


def test_max_over_ranks_single_process():
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5


def test_oracle_step_and_scenarios():
    import bench
    import gen
    import oracle
    wl, trace, prof, sp = bench.make_inputs("cfg1")
    counts, _ = oracle.bin_trace(*trace, wl.trace.window_ms, wl.trace.n_windows, gen.IN_EDGES, gen.OUT_EDGES)
    extra = bench.scenario_loads(wl, counts, 2)
    assert extra.shape == (2, 60, 9) and extra.dtype == np.float32
    n, tot = bench.oracle_step(wl, trace, prof, sp, extra)
    assert n == 3 and tot["E_total"].shape == (3,)
    # scenario s is reproducible from (seed, s) alone
    again = bench.scenario_loads(wl, counts, 1, s_begin=2)
    assert np.array_equal(again[0], extra[1])
    assert bench.scenario_loads(wl, counts, 0) is None


def test_clock_sampler_parses_rows(tmp_path):
    import bench
    cs = bench.ClockSampler.__new__(bench.ClockSampler)
    f = open(tmp_path / "c.csv", "w+")
    f.write("1965, 1965, 640.1, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n" * 3)
    f.write("1800, 1965, 990.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n")
    f.flush()
    cs.f, cs.p, cs.marks = f, None, []
    out = cs.stop()
    assert out["sm_mhz"] == 1965.0 and out["sm_max_mhz"] == 1965.0 and out["reasons"] == ["sw_power_cap"]
