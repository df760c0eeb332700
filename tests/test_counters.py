"""The recorded profiler counters (instructions, shared-memory wavefronts, DRAM bytes of the main kernels) belong to
one revision of the kernels' sources: the record carries a hash of them, the lookup marks it stale once they change,
and the committed record is that of the committed sources."""
import json
import os
import shutil

from paper_2408_00741_b200 import counters


def test_committed_counters_belong_to_the_committed_sources():
    for key in ("eval_select_kernel/cfg4", "eval_select_kernel/cfg3", "eval_select_kernel/cfg2_x256_general",
                "bin_trace_kernel/cfg3"):
        kernel, wl = key.split("/")
        rec = counters.lookup(kernel, wl)
        assert rec is not None, key
        assert not rec["stale"], f"{key}: the sources changed after the counters were taken; take them again"
        assert rec["warp_inst_per_32_evals"] > 0 and rec["command"].startswith("ncu ") and "--clock-control none" in rec["command"]
    # plausibility: the sweep executes between 5 and 8 warp instructions per 32 candidates on the threshold path,
    # the binning reads about 12 bytes per request
    assert 5.0 < counters.lookup("eval_select_kernel", "cfg4")["warp_inst_per_32_evals"] < 8.0
    assert 12.0 <= counters.lookup("bin_trace_kernel", "cfg3")["dram_bytes_per_unit"] < 13.5


def test_stale_flag_and_csv_parser(tmp_path, monkeypatch):
    csv = tmp_path / "c.csv"
    csv.write_text('==PROF== noise\n"ID","Kernel Name","Metric Name","Metric Unit","Metric Value"\n'
                   '"0","k","smsp__inst_executed.sum","inst","1,000"\n'
                   '"0","k","l1tex__data_pipe_lsu_wavefronts_mem_shared.sum","","250"\n'
                   '"0","k","dram__bytes_read.sum","Mbyte","2.5"\n"0","k","dram__bytes_write.sum","byte","500000"\n')
    m = counters.parse_csv(str(csv))
    assert m["smsp__inst_executed.sum"] == 1000.0 and m["dram__bytes_read.sum"] == 2.5e6
    pkg = tmp_path / "pkg"
    shutil.copytree(os.path.dirname(counters.__file__), pkg, ignore=shutil.ignore_patterns("*.so", "__pycache__"))
    monkeypatch.setattr(counters, "_HERE", str(pkg))
    monkeypatch.setattr(counters, "PATH", str(pkg / "counters.json"))
    rec = counters.record("bin_trace_kernel", "toy", str(csv), units=1000, evals=3200, command="ncu --clock-control none x")
    assert rec["warp_inst_per_32_evals"] == 10.0 and rec["shared_wavefronts_per_32_evals"] == 2.5
    assert rec["dram_bytes_per_unit"] == 3000.0
    assert counters.lookup("bin_trace_kernel", "toy")["stale"] is False
    with open(pkg / "csrc" / "bin_trace.cu", "a") as fh:
        fh.write("// changed\n")
    assert counters.lookup("bin_trace_kernel", "toy")["stale"] is True
    assert counters.lookup("bin_trace_kernel", "nothing") is None
    json.load(open(pkg / "counters.json"))
