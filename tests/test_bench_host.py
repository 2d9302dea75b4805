"""Host-side logic of bench.py that needs no GPU: the recorded DRAM traffic is read back per launch,
scaled by the pairs processed, and dropped when the grouped GEMM's sources have changed since the
capture; an ncu CSV log is turned into that record; the oracle sample is bounded."""
import json
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2506_07366_b200 import workloads as wl  # noqa: E402

CSV = '''==PROF== Connected to process 1
"ID","Process ID","Process Name","Host Name","Kernel Name","Context","Stream","Block Size","Grid Size","Device","CC","Section Name","Metric Name","Metric Unit","Metric Value"
"0","1","python","h","void <unnamed>::grouped_gemm_kernel<1, <unnamed>::GemmCfg<4, 2, 8, 1>>(CUtensorMap_st)","1","7","(320, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","byte","4000"
"0","1","python","h","void <unnamed>::grouped_gemm_kernel<1, <unnamed>::GemmCfg<4, 2, 8, 1>>(CUtensorMap_st)","1","7","(320, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","Kbyte","1"
"1","1","python","h","void <unnamed>::grouped_gemm_kernel<0, <unnamed>::GemmCfg<4, 2, 8, 1>>(CUtensorMap_st)","1","7","(320, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_read.sum","byte","700"
"1","1","python","h","void <unnamed>::grouped_gemm_kernel<0, <unnamed>::GemmCfg<4, 2, 8, 1>>(CUtensorMap_st)","1","7","(320, 1, 1)","(148, 1, 1)","0","10.0","Command line profiler metrics","dram__bytes_write.sum","byte","50"
'''


def test_traffic_record_roundtrip_scaling_and_invalidation(tmp_path, monkeypatch, capsys):
    log = tmp_path / "traffic.csv"
    log.write_text(CSV)
    monkeypatch.setattr(bench, "TRAFFIC_JSON", str(tmp_path / "dram_traffic.json"))
    bench.record_traffic(str(log), "mixtral_skew", 1000)
    capsys.readouterr()
    rec = json.loads((tmp_path / "dram_traffic.json").read_text())
    assert rec["gate_up"]["mixtral_skew"]["dram_read_bytes"] == 4000 and rec["gate_up"]["mixtral_skew"]["dram_write_bytes"] == 1000
    assert rec["down"]["mixtral_skew"]["dram_read_bytes"] == 700
    assert bench.recorded_traffic("mixtral_skew", 1000) == 5000           # per launch, as captured
    assert bench.recorded_traffic("mixtral_skew", 4000) == 20000          # a reduced cut, scaled by the pairs processed
    assert bench.recorded_traffic("mixtral", 1000) is None                # no capture for that workload
    monkeypatch.setattr(bench, "gemm_source_hash", lambda: "somethingelse")
    assert bench.recorded_traffic("mixtral_skew", 1000) is None           # the kernel changed since the counters were taken


def test_tracked_traffic_record_is_well_formed():
    with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
        rec = json.load(f)
    for kernel in ("gate_up", "down"):
        for wk, r in rec[kernel].items():
            assert wk in wl.WORKLOADS and r["pairs_in_capture"] > 0 and r["dram_read_bytes"] > 0 and len(r["source_hash"]) == 16


def test_oracle_sample_is_bounded_and_defaults_name_the_skewed_workload():
    for w in wl.WORKLOADS.values():
        n = bench.oracle_sample_tokens(w)
        assert 8 <= n <= w.T
        assert 6.0 * w.K * w.D * w.F * n <= 1.1e12 or n == 8             # a few seconds of fp64 work per pass
    assert bench.DEFAULT_WORKLOAD == "mixtral_skew" and "mixtral_skew" not in bench.OTHER_WORKLOADS
    w = wl.WORKLOADS[bench.DEFAULT_WORKLOAD]
    assert w.S > w.E and w.prediction == "noisy"                          # the plan really duplicates experts
