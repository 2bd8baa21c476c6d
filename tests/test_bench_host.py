"""Host-side pieces of bench.py that need no GPU: the DRAM-traffic record tied to the kernel's sources, the
clock-sample summary, the compaction of the JSON line."""
import os

import bench
from paper_2603_08343_b200 import build


def _write_record(path, digest, sources):
    with open(path, "w") as f:
        f.write("some prose about the capture\n")
        f.write(f"traffic_record: workload=training rows=65536 kernel=k<1,2> dram_bytes_read=1000 "
                f"dram_bytes_write=234 sources={','.join(sources)} sources_sha256={digest}\n")


def test_traffic_record_is_dropped_once_the_sources_change(tmp_path, monkeypatch):
    sources = ["wht_common.cuh", "misc_kernels.cuh"]
    rel = os.path.relpath(str(tmp_path / "capture.txt"), bench.ROOT)
    monkeypatch.setattr(bench, "TRAFFIC_PROFILE", rel)
    _write_record(tmp_path / "capture.txt", build.source_digest(sources), sources)
    total, where = bench.ncu_traffic("training", 65536)
    assert total == 1234 and "k<1,2>" in where
    assert bench.ncu_traffic("training", 4096)[0] is None        # no capture at that size
    assert bench.ncu_traffic("large", 65536)[0] is None          # nor for that workload
    _write_record(tmp_path / "capture.txt", "0" * 16, sources)   # the kernel has changed since
    total, where = bench.ncu_traffic("training", 65536)
    assert total is None and "stale" in where
    os.remove(tmp_path / "capture.txt")
    assert bench.ncu_traffic("training", 65536)[0] is None


def test_source_digest_depends_on_content_and_order():
    a = build.source_digest(["wht_common.cuh", "misc_kernels.cuh"])
    assert a == build.source_digest(["wht_common.cuh", "misc_kernels.cuh"]) and len(a) == 16
    assert a != build.source_digest(["misc_kernels.cuh", "wht_common.cuh"])
    assert a != build.source_digest(["wht_common.cuh"])


def test_the_committed_capture_names_files_that_exist():
    text = open(os.path.join(bench.ROOT, bench.TRAFFIC_PROFILE)).read()
    lines = [ln for ln in text.splitlines() if ln.startswith("traffic_record:")]
    assert len(lines) == 1
    rec = dict(kv.split("=", 1) for kv in lines[0].split()[1:])
    assert rec["workload"] == "training" and int(rec["rows"]) == 65536
    for name in rec["sources"].split(","):
        assert os.path.exists(os.path.join(build.CSRC, name)), name
    assert int(rec["dram_bytes_read"]) > 0 and int(rec["dram_bytes_write"]) > 0


def test_clock_summary():
    line = "0, {clk}, 1965, {w}, 0x0000000000000004, Not Active, Not Active, Not Active, {cap}"
    samples = [(10.0 + 0.02 * i, line.format(clk=1500 + i, w=990 + i, cap="Active" if i > 5 else "Not Active"))
               for i in range(20)]
    s = bench.ClockSampler.summarise(samples, 10.0, 10.2)
    assert s["samples"] == 10 and s["sm_max_mhz"] == 1965.0 and s["reasons"] == ["sw_power_cap"]
    assert 1500 <= s["sm_mhz"] <= 1512 and s["power_w_max"] == 1000.0
    assert bench.ClockSampler.summarise(samples, 50.0, 51.0)["sm_mhz"] is None
    assert bench.ClockSampler.summarise([], 0, 1)["samples"] == 0


def test_compact_rounds_floats_only():
    out = bench.compact({"a": 1.23456789, "b": [2.000004, 7], "c": {"d": "text", "e": None, "f": 123456.789}})
    assert out == {"a": 1.2346, "b": [2.0, 7], "c": {"d": "text", "e": None, "f": 123460.0}}
