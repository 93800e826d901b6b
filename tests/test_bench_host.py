"""Host-side logic of bench.py that needs no GPU."""
import hashlib
import os

import bench


def test_stored_ncu_traffic_is_reported_only_for_the_sources_it_was_taken_on(monkeypatch):
    csrc = os.path.join(os.path.dirname(os.path.abspath(bench.__file__)), "paper_2003_03477_b200", "csrc")
    sha = hashlib.sha256(open(os.path.join(csrc, "sync.cu"), "rb").read()).hexdigest()
    monkeypatch.setattr(bench, "NCU_TRAFFIC", {
        "a_kernel": {"workload": "medium", "bytes_per_launch": 123, "sources": {"sync.cu": sha}},
        "b_kernel": {"workload": "medium", "bytes_per_launch": 456, "sources": {"sync.cu": "0" * 64}},
    })
    assert bench.ncu_traffic("a_kernel", "medium") == 123
    assert bench.ncu_traffic("a_kernel", "large") is None         # another workload: other shapes
    assert bench.ncu_traffic("b_kernel", "medium") is None        # the source changed since the capture
    assert bench.ncu_traffic("c_kernel", "medium") is None        # no capture stored for it
    for name, e in bench.NCU_TRAFFIC.items():                     # what is stored names existing sources
        for src in e["sources"]:
            assert os.path.exists(os.path.join(csrc, src)), (name, src)


def test_region_statistics():
    st = bench.region_stats([10.0, 12.0, 11.0, 30.0, 10.5])
    assert st["median_ms"] == 11.0 and st["min_ms"] == 10.0 and st["max_ms"] == 30.0 and st["repeats"] == 5
    assert bench.repeats_for(region_ms=10.0, min_total_s=1.0, min_reps=10, max_reps=400) == 100
    assert bench.repeats_for(region_ms=500.0, min_total_s=1.0, min_reps=10, max_reps=400) == 10
    assert bench.repeats_for(region_ms=0.5, min_total_s=1.0, min_reps=10, max_reps=400) == 400
