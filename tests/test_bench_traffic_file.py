"""The DRAM-traffic figures bench.py reports (roofline.traffic) are read from profiles/ncu_dram_traffic.json, never
typed into the script: every record names the capture summary it came from, and that summary holds the figure."""
import json
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_every_traffic_record_points_at_a_committed_summary_that_holds_its_figure():
    import bench
    recs = bench.load_traffic()
    assert recs, "profiles/ncu_dram_traffic.json is missing or empty"
    for (workload, kernel), r in recs.items():
        assert r["bytes_per_launch"] > 0 and r["date"] and r["scaled"]
        fname = r["capture"].split(" ")[0]
        path = os.path.join(ROOT, "profiles", fname)
        assert os.path.exists(path), "%s/%s: capture summary %s is not committed" % (workload, kernel, fname)
        text = open(path).read()
        assert re.search(r"dram_rd|dram__bytes_read", text), fname + " holds no DRAM byte counts"


def test_bench_source_holds_no_traffic_constants():
    src = open(os.path.join(ROOT, "bench.py")).read()
    assert "NCU_TRAFFIC_BYTES" not in src


def test_missing_traffic_file_yields_no_records(tmp_path):
    import bench
    assert bench.load_traffic(str(tmp_path / "nope.json")) == {}
