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


def test_clock_sampler_parses_rows_and_windows(tmp_path):
    import bench
    import datetime
    cs = bench.ClockSampler.__new__(bench.ClockSampler)
    f = open(tmp_path / "c.csv", "w+")
    base = datetime.datetime(2026, 1, 2, 3, 4, 5)
    stamp = lambda k: (base + datetime.timedelta(milliseconds=100 * k)).strftime("%Y/%m/%d %H:%M:%S.%f")[:-3]
    for k in range(3):
        f.write(f"{stamp(k)}, 1965, 1965, 640.1, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n")
    f.write(f"{stamp(3)}, 1800, 1965, 990.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active\n")
    for k in range(4, 10):
        f.write(f"{stamp(k)}, 1500, 1965, 990.0, 0x0000000000000000, Not Active, Not Active, Not Active, Not Active\n")
    f.write("garbage row\n")
    f.flush()
    cs.f, cs.p = f, None
    t0 = base.timestamp()
    early = cs.window(t0, t0 + 0.2)                      # one period of slack: samples 0..3
    assert early["sm_mhz"] == 1965.0 and early["reasons"] == ["sw_power_cap"] and early["samples"] == 4
    late = cs.window(t0 + 0.6, t0 + 0.9)
    assert late["sm_mhz"] == 1500.0 and late["reasons"] == [] and late["samples"] == 5
    out = cs.stop()
    assert out["samples"] == 10 and out["sm_max_mhz"] == 1965.0 and out["reasons"] == ["sw_power_cap"]


def test_gpus_flag_starts_that_many_ranks(tmp_path):
    """`--gpus N` without a launcher: spawn_ranks starts N local ranks with the rendezvous variables set; two gloo
    ranks stand in for two GPUs, a stub stands in for the workload, rank 0 prints n_gpus = 2."""
    import bench
    import json
    import subprocess
    stub = tmp_path / "rank_stub.py"
    stub.write_text(
        "import os, sys, json\n"
        f"sys.path.insert(0, {ROOT!r})\n"
        "import torch, torch.distributed as dist\n"
        "import bench\n"
        "rank, world = int(os.environ['RANK']), int(os.environ['WORLD_SIZE'])\n"
        "assert os.environ['LOCAL_RANK'] == os.environ['RANK'] and os.environ['MASTER_ADDR'] == '127.0.0.1'\n"
        "dist.init_process_group('gloo', rank=rank, world_size=world)\n"
        "ms = bench.max_over_ranks(10.0 + rank, dist, torch.device('cpu'))\n"
        "dist.barrier()\n"
        "if rank == 0:\n"
        f"    open({str(tmp_path / 'out.json')!r}, 'w').write(json.dumps({{'n_gpus': world, 'ms': ms}}))\n"
        "dist.destroy_process_group()\n")
    assert bench.spawn_ranks(2, [sys.executable, str(stub)], timeout_s=300) == 0
    got = json.loads(open(tmp_path / "out.json").read())
    assert got == {"n_gpus": 2, "ms": 11.0}
    # a failing rank is reported
    bad = tmp_path / "bad.py"
    bad.write_text("import os, sys\nsys.exit(3 if os.environ['RANK'] == '1' else 0)\n")
    assert bench.spawn_ranks(2, [sys.executable, str(bad)], timeout_s=60) == 3
    # and the command line takes that route: --gpus 2 without WORLD_SIZE re-executes bench.py once per rank
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--help"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0
