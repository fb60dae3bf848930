"""Host-side pieces of the benchmark that need no GPU: the traffic records read from profiles/, the oracle legs."""
import os

import bench
import workloads as wl


def test_ncu_traffic_is_quoted_only_for_the_kernels_it_was_taken_on(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    os.makedirs(tmp_path / "profiles")
    os.makedirs(tmp_path / "paper_2002_05814_b200" / "csrc")
    for rel in bench.KERNEL_SOURCES:
        (tmp_path / rel).write_text("// kernel source, version 1\n")
    cur = bench.kernel_source_hash()
    (tmp_path / "profiles" / "x.md").write_text(f"text\nbench-record: workload=cfg4 kernel=reduce traffic_bytes=4.4e9 kernel_sources={cur}\n"
                                                "bench-record: workload=cfg4 kernel=fanout traffic_bytes=4.1e9 kernel_sources=0000\n")
    assert bench.ncu_traffic("cfg4", "reduce") == 4.4e9
    assert bench.ncu_traffic("cfg4", "fanout") is None          # taken on other kernels
    assert bench.ncu_traffic("cfg2", "fanout") is None          # no record
    (tmp_path / bench.KERNEL_SOURCES[0]).write_text("// kernel source, version 2\n")
    assert bench.ncu_traffic("cfg4", "reduce") is None          # the kernels have changed since


def test_committed_traffic_records_match_the_committed_kernels():
    for w, k in (("cfg4", "reduce"), ("cfg4", "fanout"), ("cfg2", "fanout"), ("cfg3", "reduce")):
        assert bench.ncu_traffic(w, k) is not None, f"profiles/ has no current record for {w} {k}: retake it or drop the line"


def test_oracle_legs_run_on_a_small_workload():
    w = wl.workload("cfg1")
    v, sample, ms = bench.oracle_sample(w, budget_s=0.2)
    assert v > 0 and "oracle" in sample
    va, cores, sample_all = bench.oracle_all_cores(w, budget_s=0.2)
    assert va > 0 and cores == len(os.sched_getaffinity(0)) and str(cores) in sample_all
    ab = bench.algorithmic_bytes(w)
    assert ab["reduce"] == 8 * (1 << 20) + (1 << 20) and ab["broadcast"] == 0
