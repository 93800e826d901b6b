"""Host-side logic of bench.py that needs no GPU."""
import hashlib
import os

import bench


def test_stored_ncu_traffic_is_reported_only_for_the_sources_it_was_taken_on():
    e = bench.NCU_TRAFFIC["gemm_tc_kernel"]
    csrc = os.path.join(os.path.dirname(os.path.abspath(bench.__file__)), "paper_2003_03477_b200", "csrc")
    unchanged = all(hashlib.sha256(open(os.path.join(csrc, n), "rb").read()).hexdigest() == h
                    for n, h in e["sources"].items())
    got = bench.ncu_traffic("gemm_tc_kernel", e["workload"])
    assert got == (e["bytes_per_launch"] if unchanged else None)
    assert bench.ncu_traffic("gemm_tc_kernel", "large") is None          # another workload: other GEMM shapes
    assert bench.ncu_traffic("embbag_fwd_kernel", e["workload"]) is None  # no capture stored for it
    assert os.path.exists(os.path.join(os.path.dirname(os.path.abspath(bench.__file__)), e["capture"]))
