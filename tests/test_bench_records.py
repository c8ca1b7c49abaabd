"""bench.py prints the decode kernel's ncu DRAM traffic only while the kernel's sources are the
ones the capture was taken on: the figure lives as a data line beside the launch-list summary
together with their hashes, and a stale figure must come out as null, not as a measurement."""
import hashlib
import json
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def test_traffic_record_is_used_only_while_the_source_hashes_match(tmp_path, monkeypatch):
    import bench

    src = "paper_2407_20485_b200/csrc/decode_step.cu"
    good = hashlib.sha256((ROOT / src).read_bytes()).hexdigest()
    rec = {"kernel": "decode_step_stream_kernel", "workload": "llama2_13b", "batch": 32,
           "dram_bytes_per_launch": 123456789, "sources": {src: good}}
    f = tmp_path / "launch_list.md"
    f.write_text("# summary\n\nbench-data: " + json.dumps(rec) + "\n")
    monkeypatch.setattr(bench, "TRAFFIC_RECORD", f)
    assert bench.ncu_decode_traffic("llama2_13b", 32) == 123456789
    assert bench.ncu_decode_traffic("llama2_13b", 4) is None          # another batch: no capture
    assert bench.ncu_decode_traffic("opt_6p7b", 32) is None
    rec["sources"][src] = "0" * 64                                     # the kernel changed since
    f.write_text("bench-data: " + json.dumps(rec) + "\n")
    assert bench.ncu_decode_traffic("llama2_13b", 32) is None
    f.write_text("no data line here\n")
    assert bench.ncu_decode_traffic("llama2_13b", 32) is None
    monkeypatch.setattr(bench, "TRAFFIC_RECORD", tmp_path / "missing.md")
    assert bench.ncu_decode_traffic("llama2_13b", 32) is None


def test_the_committed_record_names_sources_that_exist():
    import bench

    lines = [x for x in bench.TRAFFIC_RECORD.read_text().splitlines() if x.startswith("bench-data:")]
    assert len(lines) == 1
    rec = json.loads(lines[0][len("bench-data:"):])
    assert rec["kernel"] == "decode_step_stream_kernel" and rec["dram_bytes_per_launch"] > 0
    for rel in rec["sources"]:
        assert (ROOT / rel).exists(), rel
