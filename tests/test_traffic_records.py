"""Host logic of the roofline's `traffic` figure: the record an ncu capture is turned into, and bench.py's rule
for reporting it (only for the recorded workload, only while the kernel's sources hash to the recorded value)."""
import importlib
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2502_19078_b200 import ncu_summary  # noqa: E402

CSV = '''"ID","Process ID","Kernel Name","dram__bytes_read.sum","dram__bytes_write.sum"
"","","","Mbyte","Kbyte"
"0","1","void clada::sparse_ffn_kernel<__nv_bfloat16, 1, 1, 1>(FfnParams, int)","100.5","2,000"
"1","1","void clada::sparse_ffn_kernel<__nv_bfloat16, 1, 1, 1>(FfnParams, int)","99.5","4,000"
"2","1","void clada::other_kernel()","7","7"
'''


@pytest.fixture()
def sandbox(tmp_path, monkeypatch):
    (tmp_path / "profiles").mkdir()
    monkeypatch.setattr(ncu_summary, "ROOT", str(tmp_path))
    csv = tmp_path / "capture.csv"
    csv.write_text(CSV)
    return tmp_path, str(csv)


def test_record_holds_the_mean_of_the_captured_launches(sandbox):
    root, csv = sandbox
    ncu_summary.main([csv, "--kernel", "sparse_ffn_kernel", "--workload", "w1", "--units-per-launch", "2"])
    text = (root / "profiles" / "traffic_sparse_ffn_kernel.txt").read_text()
    rec = dict(l.split(": ", 1) for l in text.splitlines() if ": " in l and not l.startswith("#"))
    assert rec["launches_captured"] == "2" and rec["workload"] == "w1"
    assert float(rec["dram_bytes_read_per_unit"]) == pytest.approx(50.0e6)      # (100.5 + 99.5) MB / 2 launches / 2 units
    assert float(rec["dram_bytes_write_per_unit"]) == pytest.approx(1.5e6)      # (2000 + 4000) KB / 2 / 2
    assert float(rec["dram_bytes_per_unit"]) == pytest.approx(51.5e6)
    assert rec["sources_sha256"] == ncu_summary.sources_hash("sparse_ffn_kernel")


def test_no_matching_launch_is_an_error(sandbox):
    _, csv = sandbox
    with pytest.raises(SystemExit):
        ncu_summary.main([csv, "--kernel", "sparse_ffn_stack_kernel", "--workload", "w1"])


def test_bench_reports_a_record_only_for_its_workload_and_sources(sandbox, monkeypatch):
    root, csv = sandbox
    bench = importlib.import_module("bench")
    monkeypatch.setattr(bench, "PROFILES", str(root / "profiles"))
    ncu_summary.main([csv, "--kernel", "sparse_ffn_kernel", "--workload", "w1"])
    ncu_summary.main([csv, "--kernel", "sparse_ffn_kernel", "--workload", "w2", "--per-workload", "--units-per-launch", "4"])
    assert bench.recorded_traffic("sparse_ffn_kernel", "w1") == pytest.approx(103.0e6)
    assert bench.recorded_traffic("sparse_ffn_kernel", "w2") == pytest.approx(25.75e6)   # the per-workload record
    assert bench.recorded_traffic("sparse_ffn_kernel", "w3") is None
    assert bench.recorded_traffic("sparse_ffn_stack_kernel", "w1") is None               # no record at all
    # a record whose kernel has changed since is not reported
    monkeypatch.setattr(bench, "sources_hash", lambda kernel: "changed")
    assert bench.recorded_traffic("sparse_ffn_kernel", "w1") is None
