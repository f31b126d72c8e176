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


UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def _summary_bytes(text, section, kernel):
    """dram_rd + dram_wr of `kernel` in an ncu summary written as 'kernel: name / dram_rd value unit / dram_wr value unit'
    blocks (optionally below a '=== section' line), or in a table of 'kernel grid read write' rows (mean of its rows)."""
    if section:
        text = text[text.index("=== " + section):]
        nxt = text.find("\n=== ", 4)
        text = text if nxt < 0 else text[:nxt]
    m = re.search(r"kernel: (?:void )?%s\b.*?dram_rd\s+([0-9.]+) (\w+)\s+dram_wr\s+([0-9.]+) (\w+)" % re.escape(kernel), text, re.S)
    if m:
        return float(m.group(1)) * UNIT[m.group(2)] + float(m.group(3)) * UNIT[m.group(4)]
    rows = re.findall(r"^%s\s+\d+\s+([0-9,]+)\s+([0-9,]+)\s*$" % re.escape(kernel), text, re.M)
    assert rows, "no figures for %s" % kernel
    return sum(int(a.replace(",", "")) + int(b.replace(",", "")) for a, b in rows) / len(rows)


def test_traffic_records_match_the_figures_in_the_committed_summaries():
    recs = json.load(open(os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")))["records"]
    for r in recs:
        text = open(os.path.join(ROOT, "profiles", r["capture_file"])).read()
        got = _summary_bytes(text, r["capture_section"], r["capture_kernel"])
        assert abs(got - r["capture_bytes"]) <= 0.01 * r["capture_bytes"], (r["workload"], r["kernel"], got, r["capture_bytes"])
        assert abs(r["bytes_per_launch"] - r["capture_bytes"] * r["scale"]) <= r["scale"]


def test_bench_source_holds_no_traffic_constants():
    src = open(os.path.join(ROOT, "bench.py")).read()
    assert "NCU_TRAFFIC_BYTES" not in src


def test_missing_traffic_file_yields_no_records(tmp_path):
    import bench
    assert bench.load_traffic(str(tmp_path / "nope.json")) == {}
